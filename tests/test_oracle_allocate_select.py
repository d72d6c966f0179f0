"""Pins for the oracle's budget allocation (Sections 3.1-3.2) and its top-k / gather step."""
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _brute_allocate(S, B, w, r, L):
    """Exact rational re-statement: proportional shares with caps, then largest remainders."""
    N = len(S)
    Sq = [int(Fraction(float(s)) * (1 << 24) + Fraction(1, 2)) for s in S]      # floor(x + 1/2)
    f = w + r
    cap = L - f
    R = B - N * f
    t = [0] * N
    pool = list(range(N))
    while pool:
        tot = sum(Sq[h] for h in pool)
        if tot == 0:
            for rank, h in enumerate(pool):
                t[h] = R // len(pool) + (1 if rank < R % len(pool) else 0)
            break
        share = {h: Fraction(R * Sq[h], tot) for h in pool}
        over = [h for h in pool if share[h].__floor__() > cap]
        if over:
            for h in over:
                t[h] = cap
                pool.remove(h)
                R -= cap
            continue
        for h in pool:
            t[h] = share[h].__floor__()
        left = R - sum(t[h] for h in pool)
        order = sorted(pool, key=lambda h: (-(share[h] - t[h]), h))
        while left > 0:
            for h in order:
                if left and t[h] < cap:
                    t[h] += 1
                    left -= 1
        break
    return np.array([f + x for x in t], dtype=np.int32)


@pytest.mark.parametrize("seed", range(40))
def test_against_rational_brute_force(seed):
    rng = np.random.default_rng(seed)
    N = int(rng.integers(1, 13))
    L = int(rng.integers(8, 200))
    w = int(rng.integers(0, min(4, L)))
    r = int(rng.integers(0, 3))
    S = rng.beta(0.5, 2.0, size=N).astype(np.float32)
    if seed % 5 == 0:
        S[rng.integers(0, N)] = 0.0
    lo, hi = N * (w + r), N * L
    B = int(rng.integers(lo, hi + 1))
    b = oracle.allocate(S, B, w, r, L)
    assert np.array_equal(b, _brute_allocate(S, B, w, r, L))
    assert b.sum() == B and b.min() >= w + r and b.max() <= L


def test_floor_rule_is_a_lower_bound_when_nothing_caps():
    # w = r = 0 and no cap hit: b_h is floor(B S_h / sum S) or one more (Section 3.2's rule plus the left-over tokens).
    rng = np.random.default_rng(0)
    S = rng.uniform(0.2, 1.0, size=24).astype(np.float32)
    B, L = 2400, 1000
    b = oracle.allocate(S, B, 0, 0, L)
    Sq = np.floor(S.astype(np.float64) * 2 ** 24 + 0.5)
    fl = np.floor(B * Sq / Sq.sum()).astype(np.int64)
    assert ((b == fl) | (b == fl + 1)).all() and b.sum() == B


def test_equal_scores_give_uniform_budgets():
    # Equal head importance => the uniform (SnapKV) allocation, up to the indivisible remainder.
    b = oracle.allocate(np.full(7, 0.3, np.float32), 7 * 50 + 3, 8, 2, 400)
    assert b.max() - b.min() <= 1 and b.sum() == 353
    assert list(b) == [51, 51, 51, 50, 50, 50, 50]            # ties go to the lower head index
    b0 = oracle.allocate(np.zeros(4, np.float32), 4 * 10 + 2, 3, 0, 100)
    assert list(b0) == [11, 11, 10, 10]


def test_monotone_and_capped():
    rng = np.random.default_rng(3)
    S = rng.beta(0.5, 2.0, size=112).astype(np.float32)
    L, W = 8192, 32
    B = int(0.4 * 112 * L)
    b = oracle.allocate(S, B, W, 295, L)
    assert b.sum() == B and b.max() <= L and b.min() >= W + 295
    order = np.argsort(S, kind="stable")
    assert (np.diff(b[order]) >= 0).all()
    assert (b == L).sum() > 0                                   # this score distribution does hit the cap


def test_allocate_rejects():
    S = np.ones(4, np.float32)
    for args in [(3, 2, 0, 10), (41, 2, 0, 10), (20, 8, 4, 10)]:
        with pytest.raises(ValueError):
            oracle.allocate(S, *args)
    with pytest.raises(ValueError):
        oracle.allocate(np.array([0.5, -0.1], np.float32), 10, 1, 0, 10)
    with pytest.raises(ValueError):
        oracle.allocate(np.array([0.5, np.nan], np.float32), 10, 1, 0, 10)


@pytest.mark.parametrize("seed", range(10))
def test_select_equals_full_sort(seed):
    rng = np.random.default_rng(seed)
    P = int(rng.integers(1, 300))
    s = np.round(rng.standard_normal(P), 1)                      # many exact ties
    for k in {0, 1, P // 3, P - 1, P} & set(range(P + 1)):
        idx = oracle.select(s, k)
        want = np.sort(np.argsort(-s, kind="stable")[:k])        # score descending, lower index first among equals
        assert np.array_equal(idx, want)
        assert len(idx) == k and (np.diff(idx) > 0).all()
        if 0 < k < P:
            rest = np.setdiff1d(np.arange(P), idx)
            assert s[idx].min() >= s[rest].max()


def test_gather_copies_rows_bitwise():
    rng = np.random.default_rng(0)
    src = rng.integers(0, 65536, size=(50, 3, 8), dtype=np.uint16)     # [tok][head][d], head 1 gathered
    idx = np.array([0, 7, 8, 49], dtype=np.int32)
    out = oracle.gather(src.reshape(-1)[8:], oracle.BF16, 8, 24, idx)
    assert np.array_equal(out, src[idx, 1])
    srcf = rng.standard_normal((20, 4)).astype(np.float32)
    assert np.array_equal(oracle.gather(srcf.reshape(-1), oracle.F32, 4, 4, idx[:3]), srcf[idx[:3]])
