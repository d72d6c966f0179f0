"""GPU parity of the smoothing variants (pooling, fixed-fraction cut-off, energy cut-off without the mean), stand-alone
and inside audiokv_evict, against the oracle's akvo_smooth_variant."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06694_b200 import workloads as wl
from helpers import REL_TOL, check_kept, oracle_scores, rel_err, to_dev

pytestmark = pytest.mark.gpu

LENGTHS = [1, 2, 5, 31, 64, 257, 992, 1001, 4099, 8160, 8161, 16352, 30001]


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def _signal(rng, n):
    x = np.exp(0.5 * rng.standard_normal(n)) * 0.02
    x[0] = 3.0                                   # a sink
    return x.astype(np.float32)


@pytest.mark.parametrize("mode,param,alpha,T,pool", [
    (3, 0.0, 1.0, 0, 7), (3, 0.0, 0.5, 0, 1), (3, 0.0, 1.0, 0, 101), (4, 0.0, 1.0, 0, 7), (4, 0.0, 0.3, 0, 33),
    (1, 0.2, 1.0, 0, 1), (1, 0.5, 0.5, 4, 1), (1, 1.0, 1.0, 0, 1), (1, 0.0, 1.0, 2, 1),
    (2, 0.5, 0.5, 4, 1), (2, 0.9, 1.0, 0, 1)])
def test_smooth_variant_parity(B, mode, param, alpha, T, pool):
    W, Hkv = 8, 2
    lens = [n + W for n in LENGTHS]
    prob = B.Problem(B.AUDIOKV_BF16, 1, Hkv, Hkv, 64, lens, W, (0, 0, 0, 0), (0, 64, 0), rho=param if mode == 2 else 0.5,
                     alpha=alpha, transition_bins=T, smooth_mode=mode, smooth_kappa=param if mode == 1 else 0.0,
                     pool_kernel=pool)
    ctx = B.Context(prob)
    rng = np.random.default_rng(mode * 100 + pool)
    xs = [[_signal(rng, n) for _ in range(Hkv)] for n in LENGTHS]
    flat = np.concatenate([x for per in xs for x in per])
    scores = torch.from_numpy(flat).cuda()
    out = torch.empty_like(scores)
    kstar = torch.full((prob.total_heads,), -1, dtype=torch.int32, device="cuda")
    B.audiokv_smooth(ctx, prob, scores, out, kstar)
    torch.cuda.synchronize()
    g, gk = out.cpu().numpy(), kstar.cpu().numpy()
    off, u = 0, 0
    for n, per in zip(LENGTHS, xs):
        for x in per:
            o, ko = oracle.smooth_variant(x.astype(np.float64), mode, float(np.float32(param)), float(np.float32(alpha)),
                                          T=T, pool=pool)
            if mode == 2 and gk[u] != ko:        # fp32 transform against fp64: the cut-off may move at a near tie
                F2 = np.abs(np.fft.rfft(x.astype(np.float64))) ** 2
                F2[0] = 0.0
                E = np.cumsum(F2)
                assert abs(E[gk[u]] - param * E[-1]) / E[-1] < 2e-5 or abs(E[max(gk[u] - 1, 0)] - param * E[-1]) / E[-1] < 2e-5
                o = None
            else:
                assert gk[u] == ko, (mode, n, gk[u], ko)
            if o is not None:
                assert rel_err(g[off:off + n], o) <= REL_TOL, (mode, n)
            off += n
            u += 1
    B.audiokv_smooth(ctx, prob, scores, scores, None)      # in place
    torch.cuda.synchronize()
    assert torch.equal(scores, out)
    assert ctx.last_device_status() == 0


@pytest.mark.parametrize("over", [dict(smooth_mode=3, pool_kernel=7, alpha=1.0), dict(smooth_mode=4, pool_kernel=5, alpha=1.0),
                                  dict(smooth_mode=1, smooth_kappa=0.3, alpha=0.5),
                                  dict(smooth_mode=2, rho=0.6, alpha=0.5)])
def test_evict_with_variant(B, over):
    """The fused pass with a smoothing variant: kept sets against the oracle's steps composed by hand."""
    w = wl.generate(wl.config(1), layers=2)
    s = w.spec
    prob = B.Problem.from_workload(w, **over)
    ctx = B.Context(prob)
    TH, rows, W, L = prob.total_heads, int(w.total_budget.sum()), s.window, s.seq_lens[0]
    P = L - W
    ko = torch.zeros((rows, s.head_dim), dtype=torch.bfloat16, device="cuda")
    vo = torch.zeros_like(ko)
    kept = torch.zeros(rows, dtype=torch.int32, device="cuda")
    bud = torch.zeros(TH, dtype=torch.int32, device="cuda")
    cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
    B.audiokv_evict(ctx, prob, to_dev(w, w.q), to_dev(w, w.k), to_dev(w, w.v), torch.from_numpy(w.head_scores).cuda(),
                    [int(x) for x in w.total_budget], ko, vo, kept, bud, cu)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    sc, _ = oracle_scores(w, 0)
    budgets = oracle.allocate(w.head_scores[0].reshape(-1), int(w.total_budget[0]), W, w.base, L)
    assert np.array_equal(bud.cpu().numpy(), budgets)
    mode = over["smooth_mode"]
    param = over.get("smooth_kappa", over.get("rho", 0.0))
    cu_h, kept_h = cu.cpu().numpy(), kept.cpu().numpy()
    raw = lambda t: t.cpu().view(torch.uint16).numpy()
    for l in range(s.n_layers):
        for h in range(s.n_kv_heads):
            u = l * s.n_kv_heads + h
            sm, _ = oracle.smooth_variant(sc[l, h], mode, float(np.float32(param)), float(np.float32(over["alpha"])),
                                          T=s.transition_bins, pool=over.get("pool_kernel", 1))
            idx = kept_h[cu_h[u]:cu_h[u + 1]]
            check_kept(idx, sm, int(budgets[u]) - W, P, W, f"layer {l} head {h}")
            assert np.array_equal(raw(ko)[cu_h[u]:cu_h[u + 1]], w.k[l, h][idx])
            assert np.array_equal(raw(vo)[cu_h[u]:cu_h[u + 1]], w.v[l, h][idx])


def test_variant_rejections(B):
    w = wl.generate(wl.config(0))
    for over in (dict(smooth_mode=5), dict(smooth_mode=3, pool_kernel=4), dict(smooth_mode=3, pool_kernel=0),
                 dict(smooth_mode=1, smooth_kappa=1.5)):
        prob = B.Problem.from_workload(w, **over)
        assert B.audiokv_workspace_bytes(prob) == 0       # invalid params
