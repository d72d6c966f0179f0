"""Pins of the oracle's selection-spread statistic (the figure on the distribution of Top-K selections before and after
smoothing): numpy's histogram on the same bin rule, closed forms for flat and one-bin selections, a hand-counted case,
and selections whose histogram is known in closed form (the top of a ramp, a comb)."""
import math

import numpy as np
import pytest

import oracle


def _pack(heads):
    cu = np.concatenate([[0], np.cumsum([len(h) for h in heads])]).astype(np.int32)
    kept = np.concatenate([np.asarray(h, dtype=np.int32) for h in heads]) if cu[-1] else np.zeros(0, np.int32)
    return kept, cu


def test_hand_counted_case():
    # P = 10, 4 bins: tokens 0-2 -> bin 0, 3-4 -> bin 1, 5-7 -> bin 2, 8-9 -> bin 3 (floor(4 j / 10))
    heads = [[0, 1, 5, 10, 11], [2, 3, 9, 10, 11]]          # 10 and 11 are window tokens: not counted
    kept, cu = _pack(heads)
    hist, bal, peak = oracle.selection_spread(kept, cu, P=10, n_bins=4)
    assert hist.tolist() == [3, 1, 1, 1]
    p = np.array([3, 1, 1, 1]) / 6.0
    assert bal == pytest.approx(float(-(p * np.log(p)).sum() / math.log(4)), rel=1e-14)
    assert peak == pytest.approx(3 * 4 / 6.0, rel=1e-14)


@pytest.mark.parametrize("P,n_bins", [(1000, 10), (997, 64), (64, 64), (50, 7)])
def test_against_numpy_histogram(P, n_bins):
    rng = np.random.default_rng(P + n_bins)
    heads = [np.sort(rng.choice(P, size=rng.integers(0, P // 2), replace=False)) for _ in range(5)]
    heads = [np.concatenate([h, np.arange(P, P + 8)]) for h in heads]
    kept, cu = _pack(heads)
    hist, bal, peak = oracle.selection_spread(kept, cu, P=P, n_bins=n_bins)
    allj = np.concatenate([h[h < P] for h in heads])
    # bin edges of floor(j n / P): token j is in bin b iff b P <= j n < (b + 1) P
    edges = np.ceil(np.arange(n_bins + 1) * P / n_bins)
    want, _ = np.histogram(allj, bins=edges)
    assert hist.tolist() == want.tolist() and hist.sum() == len(allj)
    assert peak == pytest.approx(want.max() * n_bins / want.sum())
    p = want[want > 0] / want.sum()
    assert bal == pytest.approx(float(-(p * np.log(p)).sum() / math.log(n_bins)))


def test_flat_and_single_bin():
    P, n_bins = 800, 16
    flat = [np.arange(0, P, 5)]                       # 10 tokens in every bin of 50
    hist, bal, peak = oracle.selection_spread(*_pack(flat), P=P, n_bins=n_bins)
    assert set(hist.tolist()) == {10} and bal == pytest.approx(1.0, abs=1e-15) and peak == pytest.approx(1.0)
    one = [np.arange(100, 150)]                       # bin 2 alone
    hist, bal, peak = oracle.selection_spread(*_pack(one), P=P, n_bins=n_bins)
    assert hist[2] == 50 and hist.sum() == 50 and bal == 0.0 and peak == pytest.approx(16.0)
    hist, bal, peak = oracle.selection_spread(*_pack([np.arange(P, P + 4)]), P=P, n_bins=n_bins)   # window only
    assert hist.sum() == 0 and bal == 0.0 and peak == 0.0
    hist, bal, peak = oracle.selection_spread(*_pack(flat), P=P, n_bins=1)
    assert hist.tolist() == [160] and bal == 0.0 and peak == 1.0


def test_rejects_bad_arguments():
    with pytest.raises(ValueError):
        oracle.selection_spread(np.array([-1], np.int32), np.array([0, 1], np.int32), P=10, n_bins=2)
    with pytest.raises(ValueError):
        oracle.selection_spread(np.array([1], np.int32), np.array([0, 1], np.int32), P=0, n_bins=2)


def test_ramp_selection_closed_form():
    """Top-k of a rising ramp is the last k tokens: with k = two bins' worth, two bins are full and the rest empty,
    so balance = ln 2 / ln n_bins and peak = n_bins / 2; a flat-topped comb (every 8th token) is perfectly spread."""
    P, n_bins = 2048, 16
    k = 2 * P // n_bins
    ramp = oracle.select(np.arange(P, dtype=np.float64), k)
    hist, bal, peak = oracle.selection_spread(ramp, np.array([0, k], np.int32), P, n_bins)
    assert hist.tolist() == [0] * 14 + [128, 128]
    assert bal == pytest.approx(math.log(2) / math.log(16), rel=1e-14) and peak == pytest.approx(8.0)
    comb = np.zeros(P)
    comb[::8] = 1.0
    sel = oracle.select(comb, k)
    hist, bal, peak = oracle.selection_spread(sel, np.array([0, k], np.int32), P, n_bins)
    assert set(hist.tolist()) == {16} and bal == pytest.approx(1.0) and peak == pytest.approx(1.0)
