"""Head-sharded eviction on one GPU, the shards one after another: the budgets come from ONE allocation over the whole
stack (the allocation rule of Section 3.1 normalises over all layers and heads of a request), every shard of
layers then runs scoring, smoothing, selection and gather on its own with its slice of the budgets
(audiokv_evict_budgeted), and the shards' outputs put together must be what the unsharded pass gives, bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2604_06694_b200 import workloads as wl
from test_gpu_evict import check_against_oracle, run_evict

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def global_budgets(B, w_full):
    """audiokv_allocate over the whole stack; needs no K, V or Q."""
    prob = B.Problem.from_workload(w_full)
    ctx = B.Context(prob)
    TH = prob.total_heads
    budgets = torch.zeros(TH, dtype=torch.int32, device="cuda")
    cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
    B.audiokv_allocate(ctx, prob, torch.from_numpy(w_full.head_scores).cuda(), [int(x) for x in w_full.total_budget],
                       budgets, cu)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    return budgets


def run_shard(B, ws, budgets_shard):
    prob = B.Problem.from_workload(ws)
    s = ws.spec
    TH = prob.total_heads
    rows = int(budgets_shard.sum().item())
    es = ws.torch_dtype()
    k_out = torch.zeros((rows, s.head_dim), dtype=es, device="cuda")
    v_out = torch.zeros((rows, s.head_dim), dtype=es, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
    ctx = B.Context(prob)
    B.audiokv_evict_budgeted(ctx, prob, ws.as_torch(ws.q).cuda(), ws.as_torch(ws.k).cuda(), ws.as_torch(ws.v).cuda(),
                             budgets_shard, k_out, v_out, kept, cu)
    torch.cuda.synchronize()
    raw = lambda t: t.cpu().view(torch.uint16 if s.dtype == "bf16" else torch.float32).numpy()
    return dict(k_out=raw(k_out), v_out=raw(v_out), kept=kept.cpu().numpy(), cu=cu.cpu().numpy(),
                status=ctx.last_device_status())


@pytest.mark.parametrize("dtype,world", [("bf16", 2), ("bf16", 3), ("f32", 2)])
def test_layer_shards_reproduce_the_unsharded_pass(B, dtype, world):
    spec = dataclasses.replace(wl.config(1), dtype=dtype, seq_lens=(700, 1301), audio_frac=(0.8, 0.9), n_layers=4)
    full = wl.generate(spec, seed=9)
    ref = run_evict(B, full)
    if dtype == "bf16" and world == 2:
        check_against_oracle(full, ref)
    budgets = global_budgets(B, full)
    assert np.array_equal(budgets.cpu().numpy(), ref["budgets"])
    n_req, NL, Hkv = len(spec.seq_lens), spec.n_layers, spec.n_kv_heads
    seen = np.zeros(n_req * NL * Hkv, dtype=bool)
    for rank in range(world):
        l0, l1 = wl.layer_shard(NL, world, rank)
        ws = wl.generate(spec, seed=9, layer_range=(l0, l1))
        assert np.array_equal(ws.k, full.k[l0:l1]) and np.array_equal(ws.q, full.q[:, l0:l1])
        heads = wl.shard_heads(n_req, NL, Hkv, l0, l1)
        g = run_shard(B, ws, budgets[torch.from_numpy(heads).cuda()].contiguous())
        assert g["status"] == 0
        for i, u in enumerate(heads):            # shard head i is head u of the whole stack
            a, b = g["cu"][i], g["cu"][i + 1]
            ra, rb = ref["cu"][u], ref["cu"][u + 1]
            assert b - a == rb - ra
            assert np.array_equal(g["kept"][a:b], ref["kept"][ra:rb]), f"indices of head {u}"
            assert np.array_equal(g["k_out"][a:b], ref["k_out"][ra:rb]) and np.array_equal(g["v_out"][a:b], ref["v_out"][ra:rb])
            seen[u] = True
    assert seen.all()


def test_budget_outside_its_range_is_clamped_and_reported(B):
    spec = dataclasses.replace(wl.config(0), seq_lens=(300,), audio_frac=(0.8,), n_layers=1)
    w = wl.generate(spec, seed=1)
    TH = spec.n_kv_heads
    b = torch.full((TH,), 100, dtype=torch.int32, device="cuda")
    b[0] = 5          # below the window
    b[1] = 999        # above L = 300
    rows = 32 + 300 + 100 * (TH - 2)
    es = w.torch_dtype()
    prob = B.Problem.from_workload(w)
    ctx = B.Context(prob)
    k_out = torch.zeros((rows, spec.head_dim), dtype=es, device="cuda")
    v_out = torch.zeros_like(k_out)
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
    B.audiokv_evict_budgeted(ctx, prob, w.as_torch(w.q).cuda(), w.as_torch(w.k).cuda(), w.as_torch(w.v).cuda(), b, k_out,
                             v_out, kept, cu)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == B.AUDIOKV_EINVAL
    assert cu.cpu().tolist()[:3] == [0, 32, 332] and int(cu[-1]) == rows
    assert kept[:32].cpu().tolist() == list(range(268, 300)) and kept[32:332].cpu().tolist() == list(range(300))
