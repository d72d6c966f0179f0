"""Pins of the oracle's smoothing variants (pooling as in the SnapKV lineage, fixed-fraction cut-off, energy cut-off
without the mean): brute force, library routines (torch pooling, numpy FFT) and closed forms. CPU only."""
import numpy as np
import pytest
import torch

import oracle


def _rand(n, seed):
    return np.random.default_rng(seed).standard_normal(n) * 0.02 + 0.05


@pytest.mark.parametrize("n,ks", [(1, 1), (7, 3), (64, 5), (257, 7), (300, 13), (33, 33), (10, 21)])
def test_pooling_equals_brute_force_and_torch(n, ks):
    x = _rand(n, n + ks)
    h = ks // 2
    avg = np.array([sum(x[i] for i in range(j - h, j + h + 1) if 0 <= i < n) / ks for j in range(n)])
    mx = np.array([max(x[i] for i in range(j - h, j + h + 1) if 0 <= i < n) for j in range(n)])
    got_a, _ = oracle.smooth_variant(x, oracle.AVG_POOL, 0.0, 1.0, pool=ks)
    got_m, _ = oracle.smooth_variant(x, oracle.MAX_POOL, 0.0, 1.0, pool=ks)
    assert np.allclose(got_a, avg, rtol=0, atol=1e-15) and np.array_equal(got_m, mx)
    t = torch.from_numpy(x)[None, None]
    ta = torch.nn.functional.avg_pool1d(t, ks, stride=1, padding=h)[0, 0].numpy()      # zero padding counted
    tm = torch.nn.functional.max_pool1d(t, ks, stride=1, padding=h)[0, 0].numpy()
    assert np.allclose(got_a, ta, rtol=0, atol=1e-15) and np.array_equal(got_m, tm)


def test_pooling_special_cases():
    x = _rand(50, 1)
    for mode in (oracle.AVG_POOL, oracle.MAX_POOL):
        assert np.array_equal(oracle.smooth_variant(x, mode, 0.0, 1.0, pool=1)[0], x)        # window of one token
        assert np.array_equal(oracle.smooth_variant(x, mode, 0.0, 0.0, pool=9)[0], x)        # alpha = 0: no smoothing
    c = np.full(20, 0.25)
    a, _ = oracle.smooth_variant(c, oracle.AVG_POOL, 0.0, 1.0, pool=5)
    assert np.allclose(a[2:-2], 0.25) and np.isclose(a[0], 0.25 * 3 / 5) and np.isclose(a[1], 0.25 * 4 / 5)
    inc = np.arange(30, dtype=np.float64)
    m, _ = oracle.smooth_variant(inc, oracle.MAX_POOL, 0.0, 1.0, pool=7)
    assert np.array_equal(m, np.minimum(inc + 3, 29))                                       # the right edge of the window
    half, _ = oracle.smooth_variant(x, oracle.AVG_POOL, 0.0, 0.5, pool=5)
    full, _ = oracle.smooth_variant(x, oracle.AVG_POOL, 0.0, 1.0, pool=5)
    assert np.allclose(half, 0.5 * x + 0.5 * full, atol=1e-16)
    with pytest.raises(ValueError):
        oracle.smooth_variant(x, oracle.AVG_POOL, 0.0, 1.0, pool=4)                          # even window


def _numpy_lowpass(x, kstar, T):
    n = len(x)
    F = np.fft.rfft(x)
    i = np.arange(len(F))
    w = np.where(i <= kstar, 1.0, np.where(i <= kstar + T, 0.5 * (1 + np.cos(np.pi * (i - kstar) / (T + 1))), 0.0))
    return np.fft.irfft(F * w, n)


@pytest.mark.parametrize("n", [8, 9, 100, 257, 1000])
@pytest.mark.parametrize("kappa,T", [(0.0, 0), (0.2, 0), (0.5, 4), (0.8, 1), (1.0, 0)])
def test_fixed_fraction_cutoff(n, kappa, T):
    x = _rand(n, n)
    out, ks = oracle.smooth_variant(x, oracle.FIXED_FRACTION, kappa, 0.7, T=T)
    assert ks == int(np.floor(kappa * (n // 2)))
    assert np.allclose(out, 0.3 * x + 0.7 * _numpy_lowpass(x, ks, T), rtol=0, atol=1e-13)
    if kappa == 1.0:
        assert np.allclose(out, x, atol=1e-13)                       # every bin passes: identity
    if kappa == 0.0 and T == 0:
        assert np.allclose(out, 0.3 * x + 0.7 * x.mean(), atol=1e-13)  # only the mean passes
    d, kd = oracle.smooth_variant(x, oracle.FIXED_FRACTION, kappa, 0.7, T=T, direct=True)
    assert kd == ks and np.allclose(d, out, atol=1e-12)


def test_energy_cutoff_without_the_mean():
    n, f = 240, 7
    j = np.arange(n)
    for a in (0.0, 5.0, 1e3):                                       # the mean never moves the cut-off
        x = a + 0.3 * np.cos(2 * np.pi * f * j / n)
        for rho in (0.1, 0.5, 0.999):
            out, ks = oracle.smooth_variant(x, oracle.ENERGY_NO_MEAN, rho, 1.0)
            assert ks == f and np.allclose(out, x, atol=1e-9 * max(1.0, a))
    c = np.full(64, 0.5)                          # nothing but the mean (and rounding noise, which decides k*): unchanged
    out, _ = oracle.smooth_variant(c, oracle.ENERGY_NO_MEAN, 0.5, 1.0)
    assert np.allclose(out, c, atol=1e-15)
    out, ks = oracle.smooth_variant(np.zeros(64), oracle.ENERGY_NO_MEAN, 0.5, 1.0)   # exactly no energy: k* = 0
    assert ks == 0 and np.array_equal(out, np.zeros(64))
    x = _rand(501, 3)
    x -= x.mean()                                                   # zero mean: same cut-off as the method itself
    for rho in (0.2, 0.5, 0.9):
        _, k0, _ = oracle.sss(x, rho, 1.0, 0)
        o2, k2 = oracle.smooth_variant(x, oracle.ENERGY_NO_MEAN, rho, 1.0)
        assert k2 == max(k0, 1) or k2 == k0
        E = np.cumsum(np.abs(np.fft.rfft(x))[1:] ** 2)
        assert k2 == 1 + int(np.argmax(E >= rho * E[-1]))           # numpy's spectrum, bins 1..: first crossing
        assert np.allclose(o2, _numpy_lowpass(x, k2, 0), atol=1e-13)
