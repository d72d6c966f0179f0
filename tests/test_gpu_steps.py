"""GPU parity, step by step: each C entry point against the oracle on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2604_06694_b200 import workloads as wl
from helpers import KSTAR_TIE, REL_TOL, check_kept, oracle_scores, rel_err, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def _small_spec(dtype, Hq, Hkv, d, lens, W, layers=1, n_sink=1):
    return wl.WorkloadSpec(f"t_{dtype}_{Hq}_{Hkv}_{d}", dtype, layers, Hq, Hkv, d, list(lens), [0.8] * len(lens), n_sink,
                           window=W)


SCORE_CASES = [
    ("c1", lambda: wl.generate(wl.config(0))),
    ("c2_two_layers", lambda: wl.generate(wl.config(1), layers=2)),
    ("f32_d128_g1_w1", lambda: wl.generate(_small_spec("f32", 2, 2, 128, [700], 1))),
    ("bf16_d64_g7_w16_ragged", lambda: wl.generate(_small_spec("bf16", 14, 2, 64, [777, 130, 1501], 16, layers=2))),
    ("bf16_d256_g4_w32", lambda: wl.generate(_small_spec("bf16", 8, 2, 256, [1111], 32))),
    ("bf16_d128_g8_w33_short", lambda: wl.generate(_small_spec("bf16", 8, 1, 128, [34, 35, 97], 33))),
    ("bf16_d128_g7_w64", lambda: wl.generate(_small_spec("bf16", 7, 1, 128, [2100], 64))),
    # more query rows than one Q tile holds: the window is scored in chunks of rows whose column sums add up
    ("bf16_d128_g7_w48_two_chunks", lambda: wl.generate(_small_spec("bf16", 14, 2, 128, [1300, 411], 48, layers=2))),
    ("bf16_d256_g4_w64_two_chunks", lambda: wl.generate(_small_spec("bf16", 8, 2, 256, [900], 64))),
    ("bf16_d64_g8_w100_four_chunks", lambda: wl.generate(_small_spec("bf16", 8, 1, 64, [1777], 100))),
]


@pytest.mark.parametrize("name,make", SCORE_CASES, ids=[c[0] for c in SCORE_CASES])
def test_score_parity(B, name, make):
    w = make()
    prob = B.Problem.from_workload(w)
    ctx = B.Context(prob)
    q, k = to_dev(w, w.q), to_dev(w, w.k)
    scores = torch.full((B.audiokv_scores_len(prob),), float("nan"), device="cuda")
    B.audiokv_score(ctx, prob, q, k, scores)
    torch.cuda.synchronize()
    g = scores.cpu().numpy()
    assert np.isfinite(g).all()
    s = w.spec
    off = 0
    for r, L in enumerate(s.seq_lens):
        o, wm = oracle_scores(w, r)
        n = o.size
        gr = g[off:off + n].reshape(o.shape)
        off += n
        for l in range(s.n_layers):
            for h in range(s.n_kv_heads):
                assert rel_err(gr[l, h], o[l, h]) <= REL_TOL, (name, r, l, h)
        # softmax rows add up to one: prefix mass + window mass = W * G
        G = s.n_q_heads // s.n_kv_heads
        assert np.allclose(gr.sum(-1) + wm, s.window * G, rtol=2e-4)
    assert off == g.size
    assert ctx.last_device_status() == 0


def test_score_reference_jumps(B):
    """Rows whose logits jump by far more than 60 octaves in the middle of the keys, twice: every window query is the
    same vector v, and two keys far into the cache are multiples of v (4 v after 3 tiles, 9 v after 9 more), so
    their logits stand 50 and 110 nats (70 and 160 octaves) above everything before them. The running row sums of the
    first sweep must follow such jumps (the exponentials are then taken again against the new maximum), and the two
    keys end up with nearly all of the probability."""
    w = wl.generate(_small_spec("bf16", 8, 2, 128, (2048 + 64,), 32))
    d = 128
    bits = lambda x: torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).view(torch.uint16).numpy()
    v = np.ones(d, dtype=np.float32)
    v[1::2] = -1.0
    w.q[...] = bits(v)                                  # every window row and query head
    k32 = w.as_torch(w.k).to(torch.float32).numpy() * 0.05
    k32[:, :, 400, :] = 4.0 * v                         # logit 4 * 128 / sqrt(128) = 45 nats above the small keys
    k32[:, :, 1500, :] = 9.0 * v                        # and 57 nats above that one
    w.k[...] = bits(k32)
    prob = B.Problem.from_workload(w)
    ctx = B.Context(prob)
    q, k = to_dev(w, w.q), to_dev(w, w.k)
    scores = torch.full((B.audiokv_scores_len(prob),), float("nan"), device="cuda")
    B.audiokv_score(ctx, prob, q, k, scores)
    torch.cuda.synchronize()
    assert ctx.last_score_path() == "tcgen05" and ctx.last_device_status() == 0
    g = scores.cpu().numpy()
    assert np.isfinite(g).all()
    o, wm = oracle_scores(w, 0)
    s = w.spec
    P = s.seq_lens[0] - s.window
    G = s.n_q_heads // s.n_kv_heads
    gr = g.reshape(o.shape)
    for h in range(s.n_kv_heads):
        assert rel_err(gr[0, h], o[0, h]) <= REL_TOL, h
        assert abs(gr[0, h, 1500] - s.window * G) <= 1e-3 * s.window * G     # the last jump takes everything
        assert gr[0, h, 400] < 1e-20 and gr[0, h, :400].max() < 1e-30


# The long lengths, one layer each: 256 key tiles per head at L = 32768 (G = 7, so 224 query rows per head, and
# W = 64 with 448), a d = 256 head at L = 19224 (the longest request of the ragged batch), and L = 131072.
LONG_SCORE_CASES = [
    ("c3_L32768_w32", lambda: wl.generate(wl.config(2), layers=1)),
    ("c3_L32768_w64", lambda: wl.generate(dataclasses.replace(wl.config(2), window=64, n_kv_heads=2, n_q_heads=14), layers=1)),
    ("c4_L16384_sinks", lambda: wl.generate(wl.config(3), layers=1)),
    ("d256_L19224", lambda: wl.generate(dataclasses.replace(wl.config(4), seq_lens=(19224,), audio_frac=(0.9,)), layers=1)),
    ("L131072_one_head", lambda: wl.generate(dataclasses.replace(wl.config(1), seq_lens=(131072,), audio_frac=(0.9,),
                                                                 n_q_heads=7, n_kv_heads=1), layers=1)),
]


@pytest.mark.parametrize("name,make", LONG_SCORE_CASES, ids=[c[0] for c in LONG_SCORE_CASES])
def test_score_and_smooth_parity_at_full_length(B, name, make):
    """Element by element at the lengths the fused tests only see through kept sets: the scores against the oracle's,
    then audiokv_smooth on the GPU's own scores against the oracle's smoothing of the same vector."""
    w = make()
    s = w.spec
    prob = B.Problem.from_workload(w)
    ctx = B.Context(prob)
    scores = torch.full((B.audiokv_scores_len(prob),), float("nan"), device="cuda")
    B.audiokv_score(ctx, prob, to_dev(w, w.q), to_dev(w, w.k), scores)
    out = torch.empty_like(scores)
    kstar = torch.full((prob.total_heads,), -1, dtype=torch.int32, device="cuda")
    B.audiokv_smooth(ctx, prob, scores, out, kstar)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0 and ctx.last_score_path() == "tcgen05"
    g, gs, gk = scores.cpu().numpy(), out.cpu().numpy(), kstar.cpu().numpy()
    o, wm = oracle_scores(w, 0)
    P = s.seq_lens[0] - s.window
    G = s.n_q_heads // s.n_kv_heads
    worst = 0.0
    for h in range(s.n_kv_heads):
        gh = g[h * P:(h + 1) * P]
        worst = max(worst, rel_err(gh, o[0, h]))
        assert rel_err(gh, o[0, h]) <= REL_TOL, (name, h)
        assert abs(gh.sum(dtype=np.float64) + wm[0, h] - s.window * G) <= 2e-4 * s.window * G
        rho, alpha = float(np.float32(s.rho)), float(np.float32(s.alpha))
        want, ko, margin = oracle.sss(gh.astype(np.float64), rho, alpha, s.transition_bins)
        if gk[h] != ko:
            assert margin < KSTAR_TIE, (name, h, gk[h], ko, margin)
            want, _, _ = oracle.sss(gh.astype(np.float64), rho, alpha, s.transition_bins, force_kstar=int(gk[h]))
        assert rel_err(gs[h * P:(h + 1) * P], want) <= REL_TOL, (name, h)
    print(f"{name}: worst score error {worst:.2e}")


def _score_like(rng, n, kind):
    if kind == "lognormal":
        x = np.exp(rng.standard_normal(n)) * 0.02
    elif kind == "sink":
        x = np.exp(0.3 * rng.standard_normal(n)) * 0.02
        x[0] = 90.0
    else:  # smooth trend + noise
        t = np.arange(n) / max(n, 1)
        x = 0.05 + 0.03 * np.sin(7 * t) + 0.01 * rng.random(n)
    return x.astype(np.float32)


# lengths n of the smoothed sequence: tiny, primes, odd, the benchmark lengths, chirp-z in shared memory
# (prime factors above 127), and chirp-z in global scratch (large odd / large with a big prime factor)
SMOOTH_LENGTHS = [1, 2, 3, 4, 5, 7, 16, 31, 64, 97, 210, 256, 257, 510, 992, 1001, 2047, 2048, 4099, 8160, 8161,
                  12289 * 2, 16352, 32736, 32752, 32704, 30001, 32749 * 2, 65536 - 32]


@pytest.mark.parametrize("rho,alpha,T,kind", [(0.5, 0.5, 4, "sink"), (0.9, 1.0, 0, "lognormal"), (0.2, 0.3, 16, "trend"),
                                             (0.99, 0.5, 1, "sink"), (1.0, 1.0, 2, "lognormal"), (0.5, 0.0, 4, "sink")])
def test_smooth_parity(B, rho, alpha, T, kind):
    W, Hkv, NL = 8, 2, 1
    lens = [n + W for n in SMOOTH_LENGTHS]
    prob = B.Problem(B.AUDIOKV_BF16, NL, Hkv, Hkv, 64, lens, W, (0, 0, 0, 0), (0, 64, 0), rho=rho, alpha=alpha,
                     transition_bins=T)
    ctx = B.Context(prob)
    rng = np.random.default_rng(int(rho * 100) + T)
    xs = [[_score_like(rng, n, kind) for _ in range(NL * Hkv)] for n in SMOOTH_LENGTHS]
    flat = np.concatenate([x for per in xs for x in per])
    assert flat.size == B.audiokv_scores_len(prob)
    scores = torch.from_numpy(flat).cuda()
    out = torch.empty_like(scores)
    kstar = torch.full((prob.total_heads,), -1, dtype=torch.int32, device="cuda")
    B.audiokv_smooth(ctx, prob, scores, out, kstar)
    torch.cuda.synchronize()
    g, gk = out.cpu().numpy(), kstar.cpu().numpy()
    off, u, ties = 0, 0, 0
    for n, per in zip(SMOOTH_LENGTHS, xs):
        for x in per:
            o, ko, margin = oracle.sss(x.astype(np.float64), float(np.float32(rho)), float(np.float32(alpha)), T)
            if gk[u] != ko:
                # fp32 transform vs fp64: the cut-off may move only when the energy test was a near tie
                assert margin < KSTAR_TIE or rho == 1.0, (n, gk[u], ko, margin)
                o, _, _ = oracle.sss(x.astype(np.float64), float(np.float32(rho)), float(np.float32(alpha)), T,
                                     force_kstar=int(gk[u]))
                ties += 1
            assert rel_err(g[off:off + n], o) <= REL_TOL, (n, rho, alpha, T)
            off += n
            u += 1
    assert ties <= 3 or rho == 1.0
    if alpha == 0.0:
        assert np.array_equal(g, flat)          # the method without smoothing: bit-identical scores
    # in place
    B.audiokv_smooth(ctx, prob, scores, scores, None)
    torch.cuda.synchronize()
    assert np.array_equal(scores.cpu().numpy(), g)


def test_smooth_cutoff_decided_near_the_threshold(B):
    """Sequences with a known spectrum (a mean and four cosines): rho is set a thousandth below and above every value
    that the cumulative energy takes, where the cut-off must agree with the oracle exactly, and within 2e-7 of it,
    where it may move by one step only as a near tie. The cut-offs 0, 2 and 5 are settled from the first bins alone,
    9 and 14 (with T = 4) by the transform."""
    tones = {0: 0.6, 2: 1.2, 5: 0.9, 9: 0.5, 14: 0.3}
    lengths = [4096, 4099, 8160]
    energy = {k: (a * a if k == 0 else a * a / 4) for k, a in tones.items()}     # |F_k|^2 / n^2
    total = sum(energy.values())
    cum, run = [], 0.0
    for k in sorted(energy):
        run += energy[k]
        cum.append((k, run / total))
    W, T, alpha = 8, 4, 0.5
    seen, near_moves = set(), 0
    for k_at, frac in cum:
        for eps in (-1e-3, 1e-3, -2e-7, 2e-7):
            rho = frac * (1 + eps)
            if rho >= 1.0:
                continue
            prob = B.Problem(B.AUDIOKV_BF16, 1, 1, 1, 64, [n + W for n in lengths], W, (0, 0, 0, 0), (0, 64, 0),
                             rho=rho, alpha=alpha, transition_bins=T)
            ctx = B.Context(prob)
            xs = []
            for n in lengths:
                j = np.arange(n, dtype=np.float64)
                xs.append(sum(a * np.cos(2 * np.pi * k * j / n) for k, a in tones.items()).astype(np.float32))
            scores = torch.from_numpy(np.concatenate(xs)).cuda()
            out = torch.empty_like(scores)
            kstar = torch.full((prob.total_heads,), -1, dtype=torch.int32, device="cuda")
            B.audiokv_smooth(ctx, prob, scores, out, kstar)
            torch.cuda.synchronize()
            g, gk = out.cpu().numpy(), kstar.cpu().numpy()
            off = 0
            for u, (n, x) in enumerate(zip(lengths, xs)):
                r32, a32 = float(np.float32(rho)), float(np.float32(alpha))
                o, ko, margin = oracle.sss(x.astype(np.float64), r32, a32, T)
                if abs(eps) > 1e-4:
                    assert gk[u] == ko, (n, rho, gk[u], ko, margin)
                    seen.add(int(ko))
                elif gk[u] != ko:
                    assert margin < KSTAR_TIE, (n, rho, gk[u], ko, margin)
                    o, _, _ = oracle.sss(x.astype(np.float64), r32, a32, T, force_kstar=int(gk[u]))
                    near_moves += 1
                assert rel_err(g[off:off + n], o) <= REL_TOL, (n, rho)
                off += n
    assert seen == {0, 2, 5, 9, 14}, seen
    print(f"near-threshold cut-offs that moved by a tie: {near_moves}")


@pytest.mark.parametrize("seed", range(6))
def test_allocate_bit_exact(B, seed):
    rng = np.random.default_rng(seed)
    NL, Hkv = int(rng.integers(1, 30)), int(rng.integers(1, 5))
    n_req = int(rng.integers(1, 5))
    W = int(rng.integers(1, 40))
    lens = [int(rng.integers(W + 1, 5000)) for _ in range(n_req)]
    N = NL * Hkv
    base = int(rng.integers(0, max(1, (min(lens) - W) // 3)))
    S = rng.beta(0.5, 2.0, size=(n_req, NL, Hkv)).astype(np.float32)
    if seed == 1:
        S[0] = 0.0
    if seed == 2:
        S[:] = 0.25
    B_tot = [int(rng.integers(N * (W + base), N * L + 1)) for L in lens]
    if seed == 3:
        B_tot[0] = N * (W + base)
        B_tot[-1] = N * lens[-1]
    prob = B.Problem(B.AUDIOKV_BF16, NL, Hkv, Hkv, 64, lens, W, (0, 0, 0, 0), (0, 64, 0), base_per_head=base)
    ctx = B.Context(prob)
    budgets = torch.zeros(n_req * N, dtype=torch.int32, device="cuda")
    cu = torch.zeros(n_req * N + 1, dtype=torch.int32, device="cuda")
    B.audiokv_allocate(ctx, prob, torch.from_numpy(S).cuda(), B_tot, budgets, cu)
    torch.cuda.synchronize()
    g = budgets.cpu().numpy().reshape(n_req, N)
    for r in range(n_req):
        want = oracle.allocate(S[r].reshape(-1), B_tot[r], W, base, lens[r])
        assert np.array_equal(g[r], want), (seed, r)
    assert np.array_equal(cu.cpu().numpy(), np.concatenate([[0], np.cumsum(g.reshape(-1))]))
    assert ctx.last_device_status() == 0
    with pytest.raises(B.AudioKVError):
        B.audiokv_allocate(ctx, prob, torch.from_numpy(S).cuda(), [b + N * 5000 for b in B_tot], budgets, cu)


def test_allocate_config_tables(B):
    for ci in (1, 3):
        spec = wl.config(ci)
        S = np.random.Generator(np.random.Philox(key=[0, 1000])).beta(0.5, 2.0, size=(spec.n_layers, spec.n_kv_heads)).astype(np.float32)
        L, W = spec.seq_lens[0], spec.window
        N = spec.n_layers * spec.n_kv_heads
        Bt = wl.kept_total(spec, L)
        assert Bt == B.audiokv_budget_from_ratio(spec.keep, N, L, W)
        base = wl.base_per_head(spec, L)
        prob = B.Problem(B.AUDIOKV_BF16, spec.n_layers, spec.n_kv_heads, spec.n_kv_heads, 64, [L], W, (0, 0, 0, 0),
                         (0, 64, 0), base_per_head=base)
        ctx = B.Context(prob)
        budgets = torch.zeros(N, dtype=torch.int32, device="cuda")
        cu = torch.zeros(N + 1, dtype=torch.int32, device="cuda")
        B.audiokv_allocate(ctx, prob, torch.from_numpy(S).cuda(), [Bt], budgets, cu)
        assert np.array_equal(budgets.cpu().numpy(), oracle.allocate(S.reshape(-1), Bt, W, base, L))
        assert int(cu[-1]) == Bt


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64), ("bf16", 256)])
def test_select_gather_parity(B, dtype, d):
    rng = np.random.default_rng(d)
    W, Hkv, NL = 16, 2, 2
    lens = [600, 49 + W, 3000, 70000]
    spec = wl.WorkloadSpec("sg", dtype, NL, Hkv, Hkv, d, lens, [0.5] * len(lens), 0, window=W)
    w = wl.generate(dataclasses.replace(spec, seq_lens=lens[:3]))       # K/V for the first three requests only
    lens = lens[:3]
    prob = B.Problem.from_workload(w, base_per_head=0)
    ctx = B.Context(prob)
    N = NL * Hkv
    sm, bud = [], []
    for r, L in enumerate(lens):
        P = L - W
        for u in range(N):
            x = np.round(rng.standard_normal(P), 2 if u % 2 else 6).astype(np.float32)     # odd heads: many exact ties
            if u == 1:
                x[:] = 0.5                                                                 # all equal
            sm.append(x)
            bud.append([W, L, W + P // 3, W + 1][u % 4])                                    # k = 0, P, P/3, 1
    budgets = np.array(bud, dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum(budgets)]).astype(np.int32)
    rows = int(cu[-1])
    es = torch.float32 if dtype == "f32" else torch.bfloat16
    k_out = torch.zeros((rows, d), dtype=es, device="cuda")
    v_out = torch.zeros((rows, d), dtype=es, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    kd, vd = to_dev(w, w.k), to_dev(w, w.v)
    B.audiokv_select_gather(ctx, prob, torch.from_numpy(np.concatenate(sm)).cuda(), torch.from_numpy(budgets).cuda(),
                            torch.from_numpy(cu).cuda(), kd, vd, k_out, v_out, kept)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    kept = kept.cpu().numpy()
    raw = lambda t: t.cpu().view(torch.uint16 if dtype == "bf16" else torch.float32).numpy()
    ko, vo = raw(k_out), raw(v_out)
    u = 0
    for r, L in enumerate(lens):
        P = L - W
        for l in range(NL):
            for h in range(Hkv):
                idx = kept[cu[u]:cu[u + 1]]
                want = np.concatenate([oracle.select(sm[u].astype(np.float64), int(budgets[u]) - W), np.arange(P, L)])
                assert np.array_equal(idx, want), (r, l, h)           # exact fp32 inputs: ties resolve identically
                rows_k = w.k[l, h, int(w.cu_seqlen[r]):int(w.cu_seqlen[r]) + L][idx]
                rows_v = w.v[l, h, int(w.cu_seqlen[r]):int(w.cu_seqlen[r]) + L][idx]
                assert np.array_equal(ko[cu[u]:cu[u + 1]], rows_k) and np.array_equal(vo[cu[u]:cu[u + 1]], rows_v)
                u += 1


def test_score_and_gather_token_major_cache(B):
    """K and V stored [layer][token][head][d] (head stride below token stride): same scores, same kept rows."""
    w = wl.generate(wl.config(1), layers=2)
    s = w.spec
    L, Hkv, d = s.seq_lens[0], s.n_kv_heads, s.head_dim
    prob = B.Problem.from_workload(w)
    prob_t = B.Problem.from_workload(w, kv_strides=(L * Hkv * d, Hkv * d, d))
    q, k, v = to_dev(w, w.q), to_dev(w, w.k), to_dev(w, w.v)
    k_t, v_t = k.permute(0, 2, 1, 3).contiguous(), v.permute(0, 2, 1, 3).contiguous()
    out = []
    for pb, kk, vv in ((prob, k, v), (prob_t, k_t, v_t)):
        ctx = B.Context(pb)
        scores = torch.empty(B.audiokv_scores_len(pb), device="cuda")
        B.audiokv_score(ctx, pb, q, kk, scores)
        TH, rows = pb.total_heads, int(w.total_budget.sum())
        ko = torch.zeros((rows, d), dtype=torch.bfloat16, device="cuda")
        vo = torch.zeros_like(ko)
        kept = torch.zeros(rows, dtype=torch.int32, device="cuda")
        bud = torch.zeros(TH, dtype=torch.int32, device="cuda")
        cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
        B.audiokv_evict(ctx, pb, q, kk, vv, torch.from_numpy(w.head_scores).cuda(), [int(x) for x in w.total_budget],
                        ko, vo, kept, bud, cu)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == 0
        out.append((scores.cpu(), ko.cpu().view(torch.int16), vo.cpu().view(torch.int16), kept.cpu(), bud.cpu()))
    for a, b in zip(*out):
        assert torch.equal(a, b)
    o, _ = oracle_scores(w, 0)
    assert rel_err(out[1][0].numpy().reshape(o.shape)[1, 2], o[1, 2]) <= REL_TOL
