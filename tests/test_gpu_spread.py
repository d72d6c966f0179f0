"""GPU parity of audiokv_selection_spread against the oracle: histograms bit-exact, summaries to fp32 rounding."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2604_06694_b200 import workloads as wl
from test_gpu_evict import run_evict

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def spread_gpu(B, w, kept, cu, n_bins, **over):
    prob = B.Problem.from_workload(w, **over)
    ctx = B.Context(prob)
    n_req = len(w.spec.seq_lens)
    hist = torch.full((n_req, n_bins), -7, dtype=torch.int32, device="cuda")
    stats = torch.zeros((n_req, 2), dtype=torch.float32, device="cuda")
    B.audiokv_selection_spread(ctx, prob, torch.from_numpy(kept).cuda(), torch.from_numpy(cu).cuda(), n_bins, hist, stats)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    return hist.cpu().numpy(), stats.cpu().numpy()


def check(w, kept, cu, n_bins, hist, stats):
    s = w.spec
    N = s.n_layers * s.n_kv_heads
    for r, L in enumerate(s.seq_lens):
        a = cu[r * N]
        want, bal, peak = oracle.selection_spread(kept[a:cu[(r + 1) * N]], cu[r * N:(r + 1) * N + 1] - a, L - s.window,
                                                  n_bins)
        assert hist[r].tolist() == want.tolist(), f"histogram of request {r}"
        assert stats[r, 0] == pytest.approx(bal, rel=1e-5, abs=1e-6)
        assert stats[r, 1] == pytest.approx(peak, rel=1e-5, abs=1e-6)


@pytest.mark.parametrize("n_bins", [1, 7, 64, 4096])
def test_spread_of_an_eviction(B, n_bins):
    """Ragged batch, the kept indices of a real eviction; bin counts that do and do not divide the prefix."""
    spec = dataclasses.replace(wl.config(0), seq_lens=(700, 1301, 420), audio_frac=(0.8, 0.9, 0.7))
    w = wl.generate(spec, seed=4)
    g = run_evict(B, w)
    hist, stats = spread_gpu(B, w, g["kept"], g["cu"], n_bins)
    check(w, g["kept"], g["cu"], n_bins, hist, stats)
    assert hist.sum() == g["cu"][-1] - (len(g["cu"]) - 1) * spec.window      # every kept prefix token counted once


def test_spread_window_only_and_synthetic_indices(B):
    """Hand-made index lists: a request that keeps only its window (all-zero histogram and summaries), one with
    everything in a single stretch."""
    spec = dataclasses.replace(wl.config(0), seq_lens=(300, 500), audio_frac=(0.8, 0.9), n_layers=1)
    w = wl.generate(spec, seed=1)
    N, W = spec.n_kv_heads, spec.window
    heads = [np.arange(300 - W, 300) for _ in range(N)] + \
            [np.concatenate([np.arange(120, 140), np.arange(500 - W, 500)]) for _ in range(N)]
    cu = np.concatenate([[0], np.cumsum([len(h) for h in heads])]).astype(np.int32)
    kept = np.concatenate(heads).astype(np.int32)
    hist, stats = spread_gpu(B, w, kept, cu, 16)
    check(w, kept, cu, 16, hist, stats)
    assert hist[0].sum() == 0 and stats[0].tolist() == [0.0, 0.0]
    assert np.count_nonzero(hist[1]) == 1 and stats[1, 0] == 0.0 and stats[1, 1] == pytest.approx(16.0)


def test_spread_rejects_bad_bins(B):
    spec = dataclasses.replace(wl.config(0), seq_lens=(300,), audio_frac=(0.8,), n_layers=1)
    w = wl.generate(spec, seed=1)
    kept = np.zeros(8, np.int32)
    cu = np.zeros(spec.n_kv_heads + 1, np.int32)
    for nb in (0, 4097):
        with pytest.raises(B.AudioKVError) as e:
            spread_gpu(B, w, kept, cu, nb)
        assert e.value.status == B.AUDIOKV_EINVAL
