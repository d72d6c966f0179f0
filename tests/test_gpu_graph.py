"""audiokv_evict under CUDA graph capture: a serving loop records the pass once and replays it. The first call (which
uploads the plan and builds the tables) runs outside the capture; the captured call must launch the same kernels
(the allocation forks to the context's side stream and joins back) and a replay must reproduce the eager result on
new contents of the same buffers."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2604_06694_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def test_evict_captured_and_replayed(B):
    spec = dataclasses.replace(wl.config(1), seq_lens=[1301], audio_frac=[0.9])
    w1 = wl.generate(spec, seed=1, layers=3)
    w2 = wl.generate(spec, seed=2, layers=3)
    prob = B.Problem.from_workload(w1)
    ctx = B.Context(prob)
    TH, rows = prob.total_heads, int(w1.total_budget.sum())
    tb = [int(x) for x in w1.total_budget]
    q, k, v = (w1.as_torch(a).cuda() for a in (w1.q, w1.k, w1.v))
    S = torch.from_numpy(w1.head_scores).cuda()
    mk = lambda: (torch.zeros((rows, spec.head_dim), dtype=torch.bfloat16, device="cuda"),
                  torch.zeros((rows, spec.head_dim), dtype=torch.bfloat16, device="cuda"),
                  torch.zeros(rows, dtype=torch.int32, device="cuda"), torch.zeros(TH, dtype=torch.int32, device="cuda"),
                  torch.zeros(TH + 1, dtype=torch.int32, device="cuda"))
    eager = mk()
    B.audiokv_evict(ctx, prob, q, k, v, S, tb, *eager)          # also the warm-up: plan and tables go up here
    torch.cuda.synchronize()
    out = mk()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.audiokv_evict(ctx, prob, q, k, v, S, tb, *out)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    for a, b in zip(eager, out):
        assert torch.equal(a, b)
    # new contents in the same buffers: the replay must follow them
    for dst, src in ((q, w2.q), (k, w2.k), (v, w2.v)):
        dst.copy_(w2.as_torch(src).cuda())
    S.copy_(torch.from_numpy(w2.head_scores).cuda())
    graph.replay()
    torch.cuda.synchronize()
    eager2 = mk()
    B.audiokv_evict(ctx, prob, q, k, v, S, tb, *eager2)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    for a, b in zip(eager2, out):
        assert torch.equal(a, b)
    assert not torch.equal(eager[2], eager2[2])             # the two workloads really select different tokens


def test_capture_before_the_first_call_is_refused(B):
    """A call that still has to upload its plan cannot be captured: it says so and leaves the capture usable."""
    spec = dataclasses.replace(wl.config(1), seq_lens=[777], audio_frac=[0.9])
    w = wl.generate(spec, seed=1, layers=1)
    prob = B.Problem.from_workload(w)
    ctx = B.Context(prob)
    n = B.audiokv_scores_len(prob)
    q, k = w.as_torch(w.q).cuda(), w.as_torch(w.k).cuda()
    sc = torch.zeros(n, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            with pytest.raises(B.AudioKVError) as e:
                B.audiokv_score(ctx, prob, q, k, sc)
            assert e.value.status == B.AUDIOKV_ECUDA and "outside stream capture" in str(e.value)
            sc.add_(1.0)                      # the capture itself is still alive
    graph.replay()
    torch.cuda.synchronize()
    assert float(sc[0]) == 1.0
