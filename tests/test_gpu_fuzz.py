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
    heads = spec.n_layers * spec.n_kv_heads * len(spec.seq_lens)
    assert ties <= 4 * heads, (spec, ties)
