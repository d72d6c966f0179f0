"""GPU parity of the paged K/V layout: the same workload held in a pool of pages must give what the contiguous
layout gives (indices and budgets bit for bit: the arithmetic sees the same rows in the same order), and that
in turn is checked against the oracle. Pool slots that hold no token are NaN, so a reader that lets a page tail or a
foreign page through fails loudly."""
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


def run_paged(B, w, page_size, table_override=None, **over):
    k_pool, v_pool, table, n_pages, strides = wl.paged_pool(w, page_size, seed=page_size)
    if table_override is not None:
        table = table_override(table.copy(), n_pages)
    t_dev = torch.from_numpy(table).cuda()
    prob = B.Problem.from_workload(w, kv_strides=strides, kv_req_offset=None, page_size=page_size, n_pages=n_pages,
                                   page_table=t_dev, **over)
    s = w.spec
    TH = prob.total_heads
    rows = int(w.total_budget.sum())
    tb = [int(x) for x in w.total_budget]
    es = w.torch_dtype()
    k_out = torch.zeros((rows, s.head_dim), dtype=es, device="cuda")
    v_out = torch.zeros((rows, s.head_dim), dtype=es, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    budgets = torch.zeros(TH, dtype=torch.int32, device="cuda")
    cu = torch.zeros(TH + 1, dtype=torch.int32, device="cuda")
    ctx = B.Context(prob)
    B.audiokv_evict(ctx, prob, w.as_torch(w.q).cuda(), w.as_torch(k_pool).cuda(), w.as_torch(v_pool).cuda(),
                    torch.from_numpy(w.head_scores).cuda(), tb, k_out, v_out, kept, budgets, cu)
    torch.cuda.synchronize()
    raw = lambda t: t.cpu().view(torch.uint16 if s.dtype == "bf16" else torch.float32).numpy()
    return dict(k_out=raw(k_out), v_out=raw(v_out), kept=kept.cpu().numpy(), budgets=budgets.cpu().numpy(),
                cu=cu.cpu().numpy(), status=ctx.last_device_status())


def ragged(dtype, layers=2):
    spec = dataclasses.replace(wl.config(1), dtype=dtype, seq_lens=(700, 1301, 420), audio_frac=(0.8, 0.9, 0.7),
                               n_layers=layers)
    return wl.generate(spec, seed=6)


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
def test_paged_equals_contiguous_bf16(B, page_size):
    """Tensor-core scoring: tiles filled page by page; lengths that end inside a page and inside a tile."""
    w = ragged("bf16")
    ref = run_evict(B, w)
    g = run_paged(B, w, page_size)
    assert g["status"] == 0
    for key in ("budgets", "cu", "kept", "k_out", "v_out"):
        assert np.array_equal(g[key], ref[key]), key
    if page_size == 16:
        check_against_oracle(w, g)


def test_paged_equals_contiguous_f32(B):
    """fp32 inputs take the FMA scoring kernel, which follows the page table row by row."""
    w = ragged("f32", layers=1)
    ref = run_evict(B, w)
    g = run_paged(B, w, 16)
    assert g["status"] == 0
    for key in ("budgets", "cu", "kept", "k_out", "v_out"):
        assert np.array_equal(g[key], ref[key]), key
    check_against_oracle(w, g)


def test_page_id_outside_the_pool_is_reported_not_followed(B):
    """A table entry beyond the pool: the kernels report it through the status word and read no address outside the
    pool (the bad page arrives as zeros in the scoring and as page 0 in the gather)."""
    w = ragged("bf16", layers=1)

    def corrupt(table, n_pages):
        table[1, 3] = n_pages + 5
        return table

    g = run_paged(B, w, 32, table_override=corrupt)
    assert g["status"] == B.AUDIOKV_EDEVICE


def test_paged_argument_checks(B):
    w = ragged("bf16", layers=1)
    k_pool, v_pool, table, n_pages, strides = wl.paged_pool(w, 32)
    t_dev = torch.from_numpy(table).cuda()
    bad = B.Problem.from_workload(w, kv_strides=strides, page_size=48, n_pages=n_pages, page_table=t_dev)
    assert B.audiokv_scores_len(bad) == B.AUDIOKV_EUNSUPPORTED
    short = B.Problem.from_workload(w, kv_strides=strides, page_size=32, n_pages=n_pages,
                                    page_table=t_dev[:, :10].contiguous())
    assert B.audiokv_scores_len(short) == B.AUDIOKV_EINVAL
    none = B.Problem.from_workload(w, kv_strides=strides, page_size=32, n_pages=0, page_table=t_dev)
    assert B.audiokv_scores_len(none) == B.AUDIOKV_EINVAL
