"""GPU parity of audiokv_evict at the benchmark sizes: the bench workload in full (all 28 layers, the launch
configuration bench.py times), and the other configurations at their full sequence lengths and batch shapes with a
truncated layer stack so that the CPU oracle stays within seconds. Every head is compared: budgets bit-exact, kept sets
equal up to near ties, gathered K/V rows bit-exact."""
import dataclasses

import pytest

from paper_2604_06694_b200 import workloads as wl
from test_gpu_evict import check_against_oracle, run_evict

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06694_b200 import build as akv_build
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def test_config2_all_layers_as_benchmarked(B):
    w = wl.generate(wl.config(1))
    assert w.spec.n_layers == 28 and w.spec.seq_lens == [8192]
    g = run_evict(B, w)
    assert g["launches"] == 5 + 2          # the pass (5 kernels) after the two table kernels of the first call
    ties = check_against_oracle(w, g)
    # tokens exchanged at near ties over the 112 heads, and heads whose cut-off had to be handed to the oracle:
    # observed 4 to 6 and 0 (the bounds leave a margin of a few tokens, not a multiple)
    assert ties <= 16 and g["forced_kstar_heads"] == 0


@pytest.mark.parametrize("keep,W,layers", [(0.4, 32, 4), (0.2, 32, 2), (0.6, 32, 2), (0.4, 16, 2), (0.4, 64, 2)])
def test_config3_long_context_sweep(B, keep, W, layers):
    spec = dataclasses.replace(wl.config(2), keep=keep, window=W)
    w = wl.generate(spec, layers=layers)
    assert w.spec.seq_lens == [32768]
    g = run_evict(B, w)
    assert check_against_oracle(w, g) <= 16 and g["forced_kstar_heads"] == 0     # observed: up to 6 tokens, no head


def test_config4_sinks_L16k(B):
    w = wl.generate(wl.config(3), layers=6)
    assert w.spec.seq_lens == [16384] and w.spec.n_sink == 4
    g = run_evict(B, w)
    assert check_against_oracle(w, g) <= 8 and g["forced_kstar_heads"] <= 1      # observed: 2 tokens, no head


def test_config5_ragged_batch_of_eight_in_one_launch(B):
    w = wl.generate(wl.config(4), layers=3)
    assert len(w.spec.seq_lens) == 8 and min(w.spec.seq_lens) >= 2048 and max(w.spec.seq_lens) <= 32768
    g = run_evict(B, w)
    assert g["launches"] == 5 + 2
    assert check_against_oracle(w, g) <= 24 and g["forced_kstar_heads"] <= 1     # observed: 10 tokens over 48 heads, no head


def test_maximum_sequence_length(B):
    """L = 131072, the longest request the library takes: 1024 key tiles per head, a transform of 65520 complex points
    that runs block by block through global scratch, budgets up to 98 k rows per head."""
    spec = dataclasses.replace(wl.config(1), seq_lens=(131072,), audio_frac=(0.9,), n_layers=1, n_q_heads=14,
                               n_kv_heads=2)
    w = wl.generate(spec, seed=3)
    check_against_oracle(w, run_evict(B, w))
    from paper_2604_06694_b200 import binding
    too_long = binding.Problem.from_workload(w)
    too_long._seq[0] = 131073
    assert binding.audiokv_scores_len(too_long) == binding.AUDIOKV_EINVAL
