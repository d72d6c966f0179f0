"""Pins of oracle.evict_request, the composition that every fused-pass test compares with.

The paper prints no worked example, so the first case is built to be computed by hand: with
softmax scale ln 2 and keys whose only non-zero coordinate is an integer c_j, every
probability is 2^c_j / Z with an integer Z, the budgets follow from a two-head score table
with a remainder tie, and the kept sets can be read off the exponents. The second case
checks the composition (k = b - W, window append, per-head offsets, allocation floor w = W)
against the individually pinned steps and plain numpy indexing.
"""
import numpy as np

import oracle


def _tiny_case():
    L, W, d = 12, 2, 2
    c0 = np.array([3, 0, 1, 0, 2, 0, 0, 1, 0, 0, 0, 0], dtype=np.float32)   # head 0: exponent of key j
    c1 = np.array([0, 0, 0, 2, 0, 0, 1, 0, 0, 3, 1, 0], dtype=np.float32)   # head 1
    k = np.zeros((1, 2, L, d), dtype=np.float32)          # [layer][kv head][token][d]
    k[0, 0, :, 0] = c0
    k[0, 1, :, 1] = c1
    v = np.zeros_like(k)
    for j in range(L):
        v[0, 0, j] = (j, 100 + j)
        v[0, 1, j] = (200 + j, 300 + j)
    q = np.zeros((1, W, 2, d), dtype=np.float32)          # [layer][window row][query head][d]
    q[0, :, 0, 0] = 1.0
    q[0, :, 1, 1] = 1.0
    dims = (1, W, 2, 2, d, L)
    q_strides = (W * 2 * d, 2 * d, d)
    kv_strides = (2 * L * d, d, L * d)                    # layer, token, head
    return q, k, v, dims, q_strides, kv_strides, c0, c1


def test_hand_computed_request():
    q, k, v, dims, qs, kvs, c0, c1 = _tiny_case()
    L, W = 12, 2
    P = L - W
    # S = (1/4, 3/4), B = 12 rows, floor W + r = 3 per head: 6 rows to share, 1.5 and 4.5 -> 1 and 4, the left-over
    # row goes to the larger remainder, a tie here, hence to the lower head: budgets 5 and 7
    res = oracle.evict_request(q, k, v, oracle.F32, dims, qs, kvs, float(np.log(2.0)), np.array([0.25, 0.75]), 12, 1,
                               0.5, 0.0, 4)
    assert res["budgets"].tolist() == [[5, 7]]
    # window row 0 sees keys 0..10, row 1 sees 0..11; 2^c sums: head 0: 22 + 1 (+ 1), head 1: 21 + 2 (+ 1)
    want0 = 2.0 ** c0[:P].astype(np.float64) * (1 / 23 + 1 / 24)
    want1 = 2.0 ** c1[:P].astype(np.float64) * (1 / 23 + 1 / 24)
    np.testing.assert_allclose(res["scores"][0, 0], want0, rtol=1e-13)
    np.testing.assert_allclose(res["scores"][0, 1], want1, rtol=1e-13)
    np.testing.assert_array_equal(res["smoothed"], res["scores"])      # alpha = 0: no smoothing
    # head 0 keeps 3 prefix tokens: exponents 3, 2, then 1 twice (tokens 2 and 7: the lower index wins)
    assert res["kept"][0].tolist() == [0, 2, 4, 10, 11]
    # head 1 keeps 5: exponents 3, 2, 1, then two of the seven zeros (tokens 0 and 1)
    assert res["kept"][1].tolist() == [0, 1, 3, 6, 9, 10, 11]
    assert res["k_out"][0].tolist() == [[3, 0], [1, 0], [2, 0], [0, 0], [0, 0]]
    assert res["v_out"][0].tolist() == [[0, 100], [2, 102], [4, 104], [10, 110], [11, 111]]
    assert res["k_out"][1].tolist() == [[0, 0], [0, 0], [0, 2], [0, 1], [0, 3], [0, 1], [0, 0]]
    assert res["v_out"][1].tolist() == [[200, 300], [201, 301], [203, 303], [206, 306], [209, 309], [210, 310], [211, 311]]


def test_hand_computed_request_smoothed_to_the_mean():
    """alpha = 1 with a cut-off at bin 0 and no transition band leaves the mean of the sequence: every prefix token
    scores the same and the lowest indices are kept."""
    q, k, v, dims, qs, kvs, c0, _ = _tiny_case()
    k[0, 0, 0, 0] = 9.0   # the mean carries nearly all the energy: k* = 0 at rho = 0.5
    res = oracle.evict_request(q, k, v, oracle.F32, dims, qs, kvs, float(np.log(2.0)), np.array([0.25, 0.75]), 12, 1,
                               0.05, 1.0, 0)
    assert res["kstar"].tolist() == [[0, 0]]
    for h in range(2):
        np.testing.assert_allclose(res["smoothed"][0, h], res["scores"][0, h].mean(), rtol=1e-12)
    assert res["kept"][0].tolist() == [0, 1, 2, 10, 11]
    assert res["kept"][1].tolist() == [0, 1, 2, 3, 4, 10, 11]


def test_composition_from_the_pinned_steps():
    """Two layers, GQA group 2, a token-major cache with padding between heads: evict_request must equal the
    separately pinned steps put together by hand, and its gathered rows must equal numpy indexing."""
    rng = np.random.default_rng(5)
    NL, W, Hq, Hkv, d, L = 2, 3, 4, 2, 8, 41
    P = L - W
    pad = 4
    k = rng.standard_normal((NL, L, Hkv, d + pad)).astype(np.float32)   # [layer][token][kv head][d + pad]
    v = rng.standard_normal((NL, L, Hkv, d + pad)).astype(np.float32)
    q = rng.standard_normal((NL, W, Hq, d)).astype(np.float32)
    dims = (NL, W, Hq, Hkv, d, L)
    qs = (W * Hq * d, Hq * d, d)
    kvs = (L * Hkv * (d + pad), Hkv * (d + pad), d + pad)
    S = rng.uniform(0.0, 1.0, NL * Hkv).astype(np.float32)
    B, r, rho, alpha, T = 70, 2, 0.6, 0.5, 2
    scale = 0.3
    res = oracle.evict_request(q, k, v, oracle.F32, dims, qs, kvs, scale, S, B, r, rho, alpha, T)

    s, _ = oracle.score(q, k, oracle.F32, scale, qs, kvs, dims)
    np.testing.assert_array_equal(res["scores"], s)
    b = oracle.allocate(S, B, W, r, L)                     # the window is the allocation's w
    assert res["budgets"].reshape(-1).tolist() == b.tolist() and int(b.sum()) == B
    assert (b >= W + r).all() and (b <= L).all()
    for l in range(NL):
        for h in range(Hkv):
            u = l * Hkv + h
            sm, ks, _ = oracle.sss(s[l, h], rho, alpha, T)
            np.testing.assert_array_equal(res["smoothed"][l, h], sm)
            assert res["kstar"][l, h] == ks
            order = np.lexsort((np.arange(P), -sm))        # score descending, index ascending
            want = np.concatenate([np.sort(order[:b[u] - W]), np.arange(P, L)])
            assert res["kept"][u].tolist() == want.tolist()
            assert len(res["kept"][u]) == b[u]
            np.testing.assert_array_equal(res["k_out"][u], k[l, want, h, :d])
            np.testing.assert_array_equal(res["v_out"][u], v[l, want, h, :d])


def test_forced_cutoff_reaches_the_smoothing():
    """force_kstar is handed to each head's smoothing (the near-tie protocol of the GPU tests relies on it)."""
    rng = np.random.default_rng(11)
    NL, W, Hq, Hkv, d, L = 1, 2, 2, 2, 4, 30
    k = rng.standard_normal((NL, Hkv, L, d)).astype(np.float32)
    v = rng.standard_normal((NL, Hkv, L, d)).astype(np.float32)
    q = rng.standard_normal((NL, W, Hq, d)).astype(np.float32)
    dims = (NL, W, Hq, Hkv, d, L)
    qs, kvs = (W * Hq * d, Hq * d, d), (Hkv * L * d, d, L * d)
    forced = np.array([[3, 7]], dtype=np.int32)
    res = oracle.evict_request(q, k, v, oracle.F32, dims, qs, kvs, 0.5, np.ones(2), 30, 0, 0.5, 1.0, 0,
                               force_kstar=forced)
    free = oracle.evict_request(q, k, v, oracle.F32, dims, qs, kvs, 0.5, np.ones(2), 30, 0, 0.5, 1.0, 0)
    assert res["kstar"].tolist() == free["kstar"].tolist()     # the computed cut-off is still the one reported
    for h in range(2):
        assert free["kstar"][0, h] != forced[0, h]
        sm, _, _ = oracle.sss(res["scores"][0, h], 0.5, 1.0, 0, force_kstar=int(forced[0, h]))
        np.testing.assert_array_equal(res["smoothed"][0, h], sm)
        assert not np.array_equal(res["smoothed"][0, h], free["smoothed"][0, h])
        F = np.fft.rfft(res["smoothed"][0, h])
        assert np.abs(F[forced[0, h] + 1:]).max() < 1e-9 * np.abs(F[0])
