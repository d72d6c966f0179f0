"""The seeded generators: determinism, shapes, and the structure the recipe promises."""
import numpy as np
import torch

from paper_2604_06694_b200 import workloads as wl


def test_config1_shapes_and_determinism():
    a = wl.generate(wl.config(0), seed=3)
    b = wl.generate(wl.config(0), seed=3)
    c = wl.generate(wl.config(0), seed=4)
    assert a.k.shape == (1, 2, 1024, 64) and a.q.shape == (1, 1, 32, 8, 64) and a.k.dtype == np.float32
    assert np.array_equal(a.k, b.k) and np.array_equal(a.q, b.q) and np.array_equal(a.head_scores, b.head_scores)
    assert not np.array_equal(a.k, c.k)
    assert int(a.total_budget[0]) == int(0.4 * 2 * 1024)
    # the sink row has about 8x the norm of the others
    norms = np.linalg.norm(a.k[0, 0], axis=-1)
    assert 6.0 < norms[0] / norms[1:].mean() < 10.0
    # audio rows are strongly correlated with their predecessor, text rows are not
    x = a.v[0, 0]
    corr = lambda seg: np.mean(np.sum(seg[1:] * seg[:-1], -1) / 64)
    assert corr(x[:768]) > 0.85 and abs(corr(x[768:])) < 0.15


def test_ragged_bf16_layout():
    spec = wl.config(4, seed=1)
    assert len(spec.seq_lens) == 8 and all(2048 <= L <= 32768 for L in spec.seq_lens)
    import dataclasses
    small = dataclasses.replace(spec, seq_lens=[300, 77, 1500], audio_frac=[0.9, 0.8, 0.95])
    w = wl.generate(small, seed=1, layers=2)
    assert w.k.dtype == np.uint16 and w.k.shape == (2, 2, 1877, 256)
    assert list(w.cu_seqlen) == [0, 300, 377, 1877]
    assert w.as_torch(w.k).dtype == torch.bfloat16
    assert w.kv_strides() == (2 * 1877 * 256, 256, 1877 * 256)
    assert (w.head_scores >= 0).all() and (w.head_scores <= 1).all()
