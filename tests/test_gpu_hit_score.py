"""GPU parity of the offline head score (audiokv_hit_score) against the oracle: integer hit counts bit-exact,
ratios to float32 rounding; then the scores feed the budget allocation."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06694_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def _ctx(B, n_heads=4):
    prob = B.Problem(B.AUDIOKV_BF16, 1, n_heads, n_heads, 64, [64], 8, (0, 0, 0, 0), (0, 64, 0))
    return prob, B.Context(prob)


def _run(B, ctx, attn, row_len, span, K):
    H = attn.shape[1]
    counts = torch.full((H,), -1, dtype=torch.int32, device="cuda")
    s = torch.full((H,), float("nan"), device="cuda")
    B.audiokv_hit_score(ctx, torch.from_numpy(attn).cuda(), torch.from_numpy(row_len).cuda(),
                        torch.from_numpy(span).cuda(), K, counts, s)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    return counts.cpu().numpy(), s.cpu().numpy()


@pytest.mark.parametrize("n_steps,n_heads,n_audio,K", [(40, 112, 1500, 24), (7, 5, 60, 24), (12, 33, 3000, 1), (5, 8, 700, 1000)])
def test_hit_score_parity(B, n_steps, n_heads, n_audio, K):
    attn, row_len, span, _ = wl.attention_rows(n_steps, n_heads, n_audio, seed=n_steps)
    _, ctx = _ctx(B)
    gc, gs = _run(B, ctx, attn, row_len, span, K)
    s, counts = oracle.hit_score(attn, row_len, span, K)
    assert np.array_equal(gc, counts)
    assert np.array_equal(gs, s.astype(np.float32))


def test_hit_score_ties_and_short_rows(B):
    _, ctx = _ctx(B)
    attn = np.ones((3, 2, 80), dtype=np.float32)                 # all equal: the lower token index wins
    attn[1, 1, :] = np.linspace(0, 1, 80)
    row_len = np.array([80, 80, 10], dtype=np.int32)             # last row shorter than K
    span = np.array([[20, 30], [70, 79], [5, 30]], dtype=np.int32)
    gc, gs = _run(B, ctx, attn, row_len, span, 24)
    s, counts = oracle.hit_score(attn, row_len, span, 24)
    assert np.array_equal(gc, counts) and list(counts) == [4 + 0 + 5, 4 + 10 + 5]
    assert np.array_equal(gs, s.astype(np.float32))


def test_scores_feed_the_allocation(B):
    """Head scores from the statistic, summed over each KV head's query heads, drive audiokv_allocate."""
    NL, Hq, Hkv, L, W = 4, 8, 2, 2048, 32
    attn, row_len, span, _ = wl.attention_rows(30, NL * Hq, 1200, seed=9)
    prob = B.Problem(B.AUDIOKV_BF16, NL, Hq, Hkv, 64, [L], W, (0, 0, 0, 0), (0, 64, 0), base_per_head=16)
    ctx = B.Context(prob)
    gc, gs = _run(B, ctx, attn, row_len, span, 24)
    s, _ = oracle.hit_score(attn, row_len, span, 24)
    assert np.array_equal(gs, s.astype(np.float32))
    S_kv = gs.reshape(NL, Hkv, Hq // Hkv).sum(-1).astype(np.float32)      # the paper scores query heads
    Btot = B.audiokv_budget_from_ratio(0.4, NL * Hkv, L, W)
    budgets = torch.zeros(NL * Hkv, dtype=torch.int32, device="cuda")
    cu = torch.zeros(NL * Hkv + 1, dtype=torch.int32, device="cuda")
    B.audiokv_allocate(ctx, prob, torch.from_numpy(S_kv).cuda(), [Btot], budgets, cu)
    torch.cuda.synchronize()
    want = oracle.allocate(S_kv.reshape(-1), Btot, W, 16, L)
    assert np.array_equal(budgets.cpu().numpy(), want) and int(budgets.sum()) == Btot


def test_hit_score_rejections(B):
    _, ctx = _ctx(B)
    a = torch.zeros((2, 2, 16), device="cuda")
    rl = torch.full((2,), 16, dtype=torch.int32, device="cuda")
    sp = torch.zeros((2, 2), dtype=torch.int32, device="cuda")
    c = torch.zeros(2, dtype=torch.int32, device="cuda")
    s = torch.zeros(2, device="cuda")
    for k in (0, 1025):
        with pytest.raises(B.AudioKVError) as e:
            B.audiokv_hit_score(ctx, a, rl, sp, k, c, s)
        assert e.value.status == B.AUDIOKV_EINVAL
