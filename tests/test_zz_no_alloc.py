"""The allocation-free scoring entry point against the regular one and against the CPU oracle.

audiokv_score_noalloc serves callers that are not allowed to allocate device memory while they run
(a serving process whose memory pool is frozen, a plug-in without an allocator); its scratch is a
fixed array inside the library that every call on the GPU shares. This file is collected last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2604_06694_b200 import workloads as wl
from helpers import REL_TOL, oracle_scores, rel_err, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def _both(B, w):
    prob = B.Problem.from_workload(w)
    q, k = to_dev(w, w.q), to_dev(w, w.k)
    n = B.audiokv_scores_len(prob)
    ref = torch.full((n,), float("nan"), device="cuda")
    ctx = B.Context(prob)
    B.audiokv_score(ctx, prob, q, k, ref)
    got = torch.full((n,), float("nan"), device="cuda")
    B.audiokv_score_noalloc(prob, q, k, got)
    torch.cuda.synchronize()
    return got.cpu().numpy(), ref.cpu().numpy(), prob


def test_two_calls_in_a_row_match_the_regular_entry_point(B):
    # first a larger bf16 problem, then a smaller fp32 one with another shape: the second call finds the
    # first call's contents in the shared scratch and must not be affected by them
    spec = wl.WorkloadSpec("na_bf16", "bf16", 2, 14, 2, 128, [1500, 700], [0.8, 0.8], 1, window=16)
    for w in (wl.generate(spec, seed=11), wl.generate(wl.config(0), seed=12)):
        got, ref, prob = _both(B, w)
        assert np.isfinite(got).all()
        s = w.spec
        off = 0
        for r, L in enumerate(s.seq_lens):
            P = L - s.window
            want, _ = oracle_scores(w, r)              # the CPU oracle's scores of this request, fp64
            want = want.reshape(-1, P)
            for u in range(s.n_layers * s.n_kv_heads):
                assert rel_err(got[off:off + P], ref[off:off + P]) <= REL_TOL
                assert rel_err(got[off:off + P], want[u]) <= REL_TOL
                off += P
        assert off == got.size


def test_rejects_problems_beyond_the_fixed_scratch(B):
    # 48 layers x 4 heads at L = 16384 with 256 window rows needs 48 MiB of statistics: more than the 8 MiB array
    prob = B.Problem(B.AUDIOKV_BF16, 48, 32, 4, 128, [16384], 32, (0, 0, 32 * 128, 128), (4 * 16384 * 128, 128, 16384 * 128))
    x = torch.zeros(16, device="cuda")
    with pytest.raises(B.AudioKVError) as e:
        B.audiokv_score_noalloc(prob, x, x, x)
    assert e.value.status == B.AUDIOKV_EWORKSPACE
