"""GPU parity of the decode-time re-eviction (audiokv_reevict) against the oracle run head by head.

Section 3.3 lets the importance sequence come from a sliding window of decoding steps; on a compacted
cache every head has its own length, so the oracle side is the same four steps applied to each head alone:
a one-layer, one-KV-head request made of the head's own rows and its group's window queries.
"""
import dataclasses
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2604_06694_b200 import workloads as wl
from helpers import check_kept

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def make_problem(B, c, **over):
    s = c.spec
    kw = dict(dtype=B.AUDIOKV_F32 if s.dtype == "f32" else B.AUDIOKV_BF16, n_layers=s.n_layers,
              n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, seq_lens=list(s.seq_lens),
              window=s.window, q_strides=c.q_strides(), kv_strides=(0, s.head_dim, 0), rho=s.rho, alpha=s.alpha,
              transition_bins=s.transition_bins)
    kw.update(over)
    return B.Problem(**kw)


def run_reevict(B, c, budgets=None, **over):
    prob = make_problem(B, c, **over)
    s = c.spec
    budgets = c.new_budgets if budgets is None else budgets
    TH = len(budgets)
    rows = int(np.sum(budgets))
    ws = B.audiokv_reevict_workspace_bytes(prob, c.cu)
    assert ws > 0
    ctx = B.Context(prob, workspace_bytes=ws)
    es = c.torch_dtype()
    k_out = torch.zeros((rows, s.head_dim), dtype=es, device="cuda")
    v_out = torch.zeros((rows, s.head_dim), dtype=es, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
    B.audiokv_reevict(ctx, prob, c.as_torch(c.q).cuda(), c.as_torch(c.k).cuda(), c.as_torch(c.v).cuda(), c.cu, budgets,
                      k_out, v_out, kept, cu)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    raw = lambda t: t.cpu().view(torch.uint16 if s.dtype == "bf16" else torch.float32).numpy()
    return dict(k_out=raw(k_out), v_out=raw(v_out), kept=kept.cpu().numpy(), cu=cu.cpu().numpy(),
                launches=ctx.launch_count())


def check_heads(c, g, budgets=None, heads=None):
    """Every (or every listed) head against the oracle's one-head pass; rows bit-exact given the GPU's indices."""
    s = c.spec
    budgets = c.new_budgets if budgets is None else budgets
    NL, Hkv, W, d = s.n_layers, s.n_kv_heads, s.window, s.head_dim
    G = s.n_q_heads // Hkv
    dt = oracle.F32 if s.dtype == "f32" else oracle.BF16
    assert np.array_equal(g["cu"], np.concatenate([[0], np.cumsum(budgets)]))
    ties = 0
    TH = len(budgets)
    for u in (range(TH) if heads is None else heads):
        r, l, h = u // (NL * Hkv), (u // Hkv) % NL, u % Hkv
        n = int(c.cu[u + 1] - c.cu[u])
        qh = np.ascontiguousarray(c.q[r, l, :, h * G:(h + 1) * G, :])       # [W][G][d]
        kh = np.ascontiguousarray(c.k[c.cu[u]:c.cu[u + 1]])                 # [n][d]
        sc, _ = oracle.score(qh, kh, dt, 1.0 / np.sqrt(d), (0, G * d, d), (0, d, 0), (1, W, G, 1, d, n))
        sm, _, _ = oracle.sss(sc[0, 0], float(np.float32(s.rho)), float(np.float32(s.alpha)), s.transition_bins)
        a, b = g["cu"][u], g["cu"][u + 1]
        idx = g["kept"][a:b]
        ties += check_kept(idx, sm, int(budgets[u]) - W, n - W, W, f"head {u}")
        assert np.array_equal(g["k_out"][a:b], c.k[c.cu[u]:c.cu[u + 1]][idx]), f"K rows of head {u}"
        assert np.array_equal(g["v_out"][a:b], c.v[c.cu[u]:c.cu[u + 1]][idx]), f"V rows of head {u}"
    log = os.environ.get("AUDIOKV_PARITY_LOG")
    if log:
        with open(log, "a") as f:
            f.write(f"reevict {s.name} layers={NL} heads={TH} W={W} tie_tokens={ties}\n")
    return ties


def small_spec(dtype="bf16", **kw):
    base = dataclasses.replace(wl.config(1), dtype=dtype)
    return dataclasses.replace(base, **kw)


def test_reevict_bf16_two_layers(B):
    """112-head-per-request shape cut to two layers: 8 heads of different lengths, tensor-core scoring."""
    c = wl.compacted_cache(small_spec(), n_new=64, seed=3, layers=2)
    assert len(set(np.diff(c.cu).tolist())) > 4          # the heads really differ in length
    g = run_reevict(B, c)
    ties = check_heads(c, g)
    assert ties <= 4          # observed: 0


def test_reevict_f32(B):
    c = wl.compacted_cache(small_spec(dtype="f32"), n_new=40, seed=5, layers=1)
    g = run_reevict(B, c)
    assert check_heads(c, g) <= 4


def test_reevict_ragged_batch_many_heads(B):
    """More heads than one launch carries tensor maps for (3 requests x 11 layers x 4 KV heads = 132 > 120): both
    scoring sweeps and the allocation run in two launches."""
    spec = dataclasses.replace(wl.config(1), seq_lens=(700, 1301, 420), audio_frac=(0.8, 0.9, 0.7), n_layers=11)
    c = wl.compacted_cache(spec, n_new=33, seed=11)
    assert len(c.new_budgets) == 132
    g = run_reevict(B, c)
    assert g["launches"] == 2 + 3 + 4 + 1 + 1      # tables, allocation x3 (64 requests each), sweeps x2 x2, smoothing, gather
    assert check_heads(c, g) <= 6      # observed: 0 over 112 to 132 heads


def test_reevict_keep_all_and_window_only(B):
    """Degenerate budgets: a head that keeps everything, one that keeps its window alone."""
    c = wl.compacted_cache(small_spec(), n_new=16, seed=7, layers=1)
    n = np.diff(c.cu)
    budgets = c.new_budgets.copy()
    budgets[0] = n[0]
    budgets[1] = c.spec.window
    g = run_reevict(B, c, budgets=budgets)
    check_heads(c, g, budgets=budgets)
    a, b = g["cu"][0], g["cu"][1]
    assert np.array_equal(g["kept"][a:b], np.arange(n[0]))
    a, b = g["cu"][1], g["cu"][2]
    assert np.array_equal(g["kept"][a:b], np.arange(n[1] - c.spec.window, n[1]))


def test_reevict_rejects_bad_arguments(B):
    c = wl.compacted_cache(small_spec(), n_new=16, seed=7, layers=1)
    bad = c.new_budgets.copy()
    bad[2] = c.spec.window - 1
    with pytest.raises(B.AudioKVError) as e:
        run_reevict(B, c, budgets=bad)
    assert e.value.status == B.AUDIOKV_EINVAL
    bad = c.new_budgets.copy()
    bad[2] = int(np.diff(c.cu)[2]) + 1
    with pytest.raises(B.AudioKVError) as e:
        run_reevict(B, c, budgets=bad)
    assert e.value.status == B.AUDIOKV_EINVAL
    prob = make_problem(B, c)
    cu = c.cu.copy()
    cu[0] = 1
    assert B.audiokv_reevict_workspace_bytes(prob, cu) == 0


def test_q_req_offset_matches_stride(B):
    """audiokv_score with explicit per-request query offsets equals the strided layout, also when permuted."""
    spec = dataclasses.replace(wl.config(1), seq_lens=(500, 900), audio_frac=(0.8, 0.9), n_layers=2)
    w = wl.generate(spec, seed=2)
    prob = B.Problem.from_workload(w)
    n = B.audiokv_scores_len(prob)
    ctx = B.Context(prob)
    q, k = w.as_torch(w.q).cuda(), w.as_torch(w.k).cuda()
    ref = torch.zeros(n, dtype=torch.float32, device="cuda")
    B.audiokv_score(ctx, prob, q, k, ref)
    # the two requests' queries swapped in memory, the offsets pointing at the swapped places
    q_sw = torch.stack([q[1], q[0]]).contiguous()
    st = w.q_strides()[0]
    prob2 = B.Problem.from_workload(w, q_req_offset=[st, 0])
    got = torch.zeros(n, dtype=torch.float32, device="cuda")
    B.audiokv_score(ctx, prob2, q_sw, k, got)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    assert torch.equal(ref, got)


def test_reevict_full_size_sampled_heads(B):
    """The 7B shape at L = 8192 after one eviction and 128 decoded tokens: 112 heads of 1.8k to 5k rows (one
    transform plan per distinct length); sampled heads against the oracle, and for
    every head the properties that hold at any size."""
    c = wl.compacted_cache(wl.config(1), n_new=128, seed=1)
    assert len(c.new_budgets) == 112
    g = run_reevict(B, c)
    assert check_heads(c, g, heads=[0, 17, 44, 63, 64, 111]) <= 6
    W = c.spec.window
    for u in range(112):
        a, b = g["cu"][u], g["cu"][u + 1]
        n = int(c.cu[u + 1] - c.cu[u])
        idx = g["kept"][a:b]
        assert b - a == c.new_budgets[u]
        assert (np.diff(idx) > 0).all() and idx[0] >= 0 and np.array_equal(idx[-W:], np.arange(n - W, n))
        assert np.array_equal(g["k_out"][a:b], c.k[c.cu[u]:c.cu[u + 1]][idx])
        assert np.array_equal(g["v_out"][a:b], c.v[c.cu[u]:c.cu[u + 1]][idx])
