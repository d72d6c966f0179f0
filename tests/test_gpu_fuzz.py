"""Seeded random shapes through the whole pass: head counts, head dimension, window, group size, lengths (even, odd,
prime), ragged batches, element type, retention ratio and smoothing parameters drawn at random; every case against the
oracle with the usual tolerances. The draws are fixed by the seed, so a failure names its case."""
import dataclasses

import numpy as np
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


def draw(case: int):
    rng = np.random.default_rng(1000 + case)
    hkv = int(rng.choice([1, 2, 4]))
    g = int(rng.choice([1, 2, 4, 7, 8]))
    w = int(rng.choice([8, 16, 32]))
    n_req = int(rng.choice([1, 1, 2, 3]))
    lens = [int(rng.integers(w + 40, 1800)) for _ in range(n_req)]
    if case % 3 == 0:
        lens[0] = [509 + w, 1021 + w, 1499 + w][case // 3 % 3]          # prime prefix lengths: chirp-z
    return dataclasses.replace(
        wl.config(1), dtype=str(rng.choice(["bf16", "bf16", "f32"])), n_layers=int(rng.integers(1, 4)),
        n_q_heads=hkv * g, n_kv_heads=hkv, head_dim=int(rng.choice([64, 128, 256])), seq_lens=lens,
        audio_frac=[float(rng.uniform(0.5, 0.95)) for _ in lens], n_sink=int(rng.choice([0, 1, 4])), window=w,
        keep=float(rng.choice([0.2, 0.4, 0.6, 0.8])), rho=float(rng.choice([0.3, 0.5, 0.9, 0.99])),
        alpha=float(rng.choice([0.25, 0.5, 1.0])), transition_bins=int(rng.choice([0, 2, 4, 8])))


@pytest.mark.parametrize("case", range(40))
def test_random_shape(B, case):
    spec = draw(case)
    w = wl.generate(spec, seed=case)
    g = run_evict(B, w)
    ties = check_against_oracle(w, g)
    # observed over the 40 cases: no token exchanged at a near tie, one head in one case with a moved cut-off
    assert ties <= 4 and g["forced_kstar_heads"] <= 2, (spec, ties, g["forced_kstar_heads"])


@pytest.mark.parametrize("case", range(12))
def test_random_shape_paged(B, case):
    """The same draws with K and V in a pool of pages of a random size (bf16 and fp32): identical to the contiguous run."""
    from test_gpu_paged import run_paged
    spec = draw(100 + case)
    w = wl.generate(spec, seed=case)
    ref = run_evict(B, w)
    g = run_paged(B, w, int(np.random.default_rng(case).choice([16, 32, 64, 128])))
    assert g["status"] == 0
    for key in ("budgets", "cu", "kept", "k_out", "v_out"):
        assert np.array_equal(g[key], ref[key]), key


@pytest.mark.parametrize("case", range(12))
def test_random_shape_reevict(B, case):
    """Random compacted caches (per-head lengths, decoded tokens, element type) against the oracle head by head."""
    from test_gpu_reevict import check_heads, run_reevict
    spec = draw(200 + case)
    rng = np.random.default_rng(case)
    c = wl.compacted_cache(spec, n_new=int(rng.integers(spec.window, 200)), seed=case, spread=float(rng.uniform(0.0, 0.8)))
    g = run_reevict(B, c)
    assert check_heads(c, g) <= 4 * len(c.new_budgets)
