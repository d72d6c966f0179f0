"""A bounded wait that runs out: the scoring kernel must report it and leave the context usable.

Nothing is injected and nothing is skipped: the limit of the kernels' waits is set to one clock cycle, so the first
wait that finds its barrier not yet complete (the tensor-core warp waiting for the first copy of Q, for one) gives up.
The CTA then stops the ordinary way: it waits, with the stop path's own limit, for its copies and tensor-core operations
in flight, releases its tensor memory and the kernel writes AUDIOKV_ETIMEOUT. The same context then scores the same
inputs with the default limit and must agree with the oracle.
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


def test_wait_limit_runs_out_then_the_context_recovers(B):
    spec = wl.WorkloadSpec("timeout_case", "bf16", 1, 4, 1, 128, [1000], [0.8], 1, window=16)   # one head, 8 key tiles
    w = wl.generate(spec, seed=2)
    prob = B.Problem.from_workload(w)
    ctx = B.Context(prob)
    q, k = to_dev(w, w.q), to_dev(w, w.k)
    n = B.audiokv_scores_len(prob)
    scores = torch.zeros(n, device="cuda")
    B.audiokv_score(ctx, prob, q, k, scores)           # uploads the plan; the ordinary result
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    want, _ = oracle_scores(w, 0)
    assert rel_err(scores.cpu().numpy(), want[0, 0]) <= REL_TOL

    default = B.audiokv_set_wait_limit(1)
    try:
        assert default > 10**8
        junk = torch.zeros(n, device="cuda")
        B.audiokv_score(ctx, prob, q, k, junk)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == B.AUDIOKV_ETIMEOUT
        assert ctx.last_device_status() == 0           # reported once
    finally:
        assert B.audiokv_set_wait_limit(0) == 1        # back to the default
    assert B.audiokv_set_wait_limit(0) == default

    again = torch.zeros(n, device="cuda")
    for _ in range(2):
        B.audiokv_score(ctx, prob, q, k, again)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    assert np.array_equal(again.cpu().numpy(), scores.cpu().numpy())
