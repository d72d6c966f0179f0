"""Pins for the oracle's Spectral Score Smoothing (Section 3.3) and its DFT routines."""
import math

import numpy as np
import pytest

import oracle


def _sizes():
    # every n up to 512: all primes, prime powers, odd and even lengths in that range
    return list(range(1, 513))


@pytest.mark.parametrize("n", _sizes())
def test_fast_dft_equals_definition_and_numpy(n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal(n)
    Fd = oracle.rfft(x, direct=True)
    Ff = oracle.rfft(x, direct=False)
    Fn = np.fft.rfft(x)
    tol = 1e-12 * max(1.0, np.abs(Fn).max())
    assert np.abs(Fd - Fn).max() < tol and np.abs(Ff - Fn).max() < tol
    for direct in (True, False):
        assert np.abs(oracle.irfft(Fn, n, direct=direct) - np.fft.irfft(Fn, n)).max() < 1e-12 * max(1.0, np.abs(x).max())


def test_dft_of_a_shifted_impulse():
    # x = delta_{j0}  =>  F_k = exp(-2 pi i j0 k / n): catches a wrong sign or a transposed index.
    n, j0 = 45, 7
    x = np.zeros(n)
    x[j0] = 1.0
    k = np.arange(n // 2 + 1)
    want = np.exp(-2j * np.pi * j0 * k / n)
    assert np.abs(oracle.rfft(x) - want).max() < 1e-14
    assert np.abs(oracle.rfft(x, direct=True) - want).max() < 1e-14


# the prefix lengths of the workloads: L - 32 for L = 8192, 1024, 16384, 32768 (W = 16, 32), and the ragged batch's
# lengths (among them the odd prime 15227 and lengths with a large prime factor), plus a prime above 4096
@pytest.mark.parametrize("n", [8160, 992, 4099, 16352, 32736, 32752, 11536, 8572, 15227, 4753, 19192, 5644, 9081, 11878])
def test_full_size_fast_dft_against_numpy(n):
    x = np.random.default_rng(0).standard_normal(n)
    F = np.fft.rfft(x)
    assert np.abs(oracle.rfft(x) - F).max() < 1e-9
    assert np.abs(oracle.irfft(F, n) - x).max() < 1e-11


@pytest.mark.parametrize("n", [31, 32, 257, 600])
@pytest.mark.parametrize("direct", [True, False])
def test_identity_at_full_passband_and_at_alpha_zero(n, direct):
    x = np.random.default_rng(n).random(n)
    out, kstar, _ = oracle.sss(x, 1.0, 1.0, 0, direct=direct)
    assert np.abs(out - x).max() < 1e-12
    out, _, _ = oracle.sss(x, 1.0, 1.0, 5, direct=direct)       # the band lies after k*: still the identity
    assert np.abs(out - x).max() < 1e-12
    out, _, _ = oracle.sss(x, 0.5, 0.0, 4, direct=direct)       # alpha = 0: the method without smoothing
    assert np.array_equal(out, x)


@pytest.mark.parametrize("n", [1, 2, 3, 50, 51])
def test_constant_vector_unchanged(n):
    x = np.full(n, 0.37)
    for T in (0, 3):
        out, kstar, _ = oracle.sss(x, 0.5, 1.0, T)
        assert kstar == 0
        assert np.abs(out - x).max() < 1e-14


def test_single_cosine_closed_form():
    # x_j = a + b cos(2 pi f j / n): m_0^2 = (n a)^2, m_f^2 = (n b / 2)^2, nothing else.
    # k* = 0 iff rho <= a^2 / (a^2 + b^2/4), else k* = f; output is the mean, resp. x itself.
    n, f, a, b = 120, 9, 1.0, 1.6
    j = np.arange(n)
    x = a + b * np.cos(2 * np.pi * f * j / n)
    share = a * a / (a * a + b * b / 4)
    out, kstar, _ = oracle.sss(x, share - 0.05, 1.0, 0)
    assert kstar == 0 and np.abs(out - a).max() < 1e-12
    out, kstar, _ = oracle.sss(x, share + 0.05, 1.0, 0)
    assert kstar == f and np.abs(out - x).max() < 1e-12
    out, kstar, _ = oracle.sss(x, share - 0.05, 0.25, 0)
    assert np.abs(out - (0.75 * x + 0.25 * a)).max() < 1e-12
    _, _, _, E = oracle.sss(x, 0.5, 1.0, 0, want_energy=True)
    assert np.isclose(E[0], (n * a) ** 2) and np.isclose(E[f] - E[f - 1], (n * b / 2) ** 2) and np.isclose(E[-1], E[f])


def test_two_tones_with_transition_band():
    # Tones at f1 < f2; rho puts k* at f1, and f2 = f1 + 2 falls in a T = 3 band: its weight is (1 + cos(2 pi / 4)) / 2 = 1/2.
    n, f1, f2 = 96, 5, 7
    j = np.arange(n)
    c1 = np.cos(2 * np.pi * f1 * j / n)
    c2 = np.cos(2 * np.pi * f2 * j / n + 0.3)
    x = 2.0 * c1 + 1.0 * c2                                   # energies: f1 -> (n)^2, f2 -> (n/2)^2
    out, kstar, _ = oracle.sss(x, 0.7, 1.0, 3)
    assert kstar == f1
    assert np.abs(out - (2.0 * c1 + 0.5 * c2)).max() < 1e-12
    out, _, _ = oracle.sss(x, 0.7, 1.0, 1)                     # band of one bin: f2 is cut
    assert np.abs(out - 2.0 * c1).max() < 1e-12
    out, _, _ = oracle.sss(x, 0.7, 1.0, 0)                     # the paper's binary mask
    assert np.abs(out - 2.0 * c1).max() < 1e-12


def test_taper_weights_via_impulse():
    # For an impulse every |F_k| = 1, so E(k) = k + 1 and k* = ceil(rho (Kb + 1)) - 1; the output's spectrum is the mask itself.
    n, T, rho = 64, 4, 0.5
    x = np.zeros(n)
    x[0] = 1.0
    out, kstar, _ = oracle.sss(x, rho, 1.0, T)
    Kb = n // 2
    assert kstar == math.ceil(rho * (Kb + 1)) - 1
    w = np.fft.rfft(out).real
    want = np.zeros(Kb + 1)
    want[: kstar + 1] = 1.0
    for i in range(1, T + 1):
        want[kstar + i] = 0.5 * (1 + math.cos(math.pi * i / (T + 1)))
    assert np.abs(w - want).max() < 1e-13
    assert np.abs(np.fft.rfft(out).imag).max() < 1e-13


@pytest.mark.parametrize("n", [63, 64])
def test_invariants(n):
    rng = np.random.default_rng(n)
    x = rng.random(n) + 0.1 * np.sin(np.arange(n) / 3.0)
    out, kstar, _, E = oracle.sss(x, 0.9, 0.6, 2, want_energy=True)
    assert 0 < kstar < n // 2
    # mean preservation (w_0 = 1)
    assert np.isclose(out.sum(), x.sum(), rtol=1e-13)
    # scale equivariance and shift equivariance (magnitudes are shift-invariant => same k*)
    out2, k2, _ = oracle.sss(3.5 * x, 0.9, 0.6, 2)
    assert k2 == kstar and np.allclose(out2, 3.5 * out, rtol=1e-12)
    out3, k3, _ = oracle.sss(np.roll(x, 11), 0.9, 0.6, 2)
    assert k3 == kstar and np.allclose(out3, np.roll(out, 11), atol=1e-13)
    # Parseval for the one-sided sum: 2 E(Kb) - m_0^2 - [n even] m_{n/2}^2 = n sum x^2
    F = np.fft.rfft(x)
    lhs = 2 * E[-1] - abs(F[0]) ** 2 - (abs(F[-1]) ** 2 if n % 2 == 0 else 0.0)
    assert np.isclose(lhs, n * (x ** 2).sum(), rtol=1e-12)
    assert np.allclose(E, np.cumsum(np.abs(F) ** 2), rtol=1e-12)
    # with the binary mask the filter is a projection: filtering twice at the same k* changes nothing
    lp, _, _ = oracle.sss(x, 0.9, 1.0, 0)
    lp2, _, _ = oracle.sss(lp, 0.9, 1.0, 0, force_kstar=kstar)
    assert np.abs(lp2 - lp).max() < 1e-13


@pytest.mark.parametrize("n,rho,alpha,T", [(300, 0.2, 0.5, 4), (301, 0.5, 1.0, 16), (128, 0.8, 0.5, 1), (77, 0.99, 0.3, 0)])
def test_against_numpy_pipeline(n, rho, alpha, T):
    # The same steps with numpy's FFT as the transform (an independent library routine for both directions).
    rng = np.random.default_rng(n)
    x = rng.random(n) ** 3
    F = np.fft.rfft(x)
    E = np.cumsum(np.abs(F) ** 2)
    kstar = int(np.argmax(E >= rho * E[-1]))
    i = np.arange(n // 2 + 1)
    w = np.where(i <= kstar, 1.0, np.where(i <= kstar + T, 0.5 * (1 + np.cos(np.pi * (i - kstar) / (T + 1))), 0.0))
    want = (1 - alpha) * x + alpha * np.fft.irfft(F * w, n)
    for direct in (True, False):
        out, k, _ = oracle.sss(x, rho, alpha, T, direct=direct)
        assert k == kstar
        assert np.abs(out - want).max() < 1e-13


def test_zero_input_and_forced_cutoff():
    out, kstar, _ = oracle.sss(np.zeros(10), 0.5, 1.0, 2)
    assert kstar == 0 and np.array_equal(out, np.zeros(10))
    x = np.random.default_rng(0).random(40)
    a, k, _ = oracle.sss(x, 0.9, 1.0, 0)
    b, k_reported, _ = oracle.sss(x, 0.1, 1.0, 0, force_kstar=k)
    assert np.array_equal(a, b)          # the forced cut-off decides the mask ...
    assert k_reported <= k                # ... while the computed one (rho = 0.1) is still reported
