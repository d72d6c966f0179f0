"""Pins of the oracle's offline head score (top-K of attention rows against word spans): brute force, numpy's stable
sort, closed forms. CPU only."""
import numpy as np

import oracle
from paper_2604_06694_b200 import workloads as wl


def test_against_numpy_stable_sort_and_brute_force():
    attn, row_len, span, _ = wl.attention_rows(n_steps=9, n_heads=5, n_audio=200, seed=3)
    K = 24
    s, counts = oracle.hit_score(attn, row_len, span, K)
    for a in range(attn.shape[1]):
        tot, mean = 0, 0.0
        for t in range(attn.shape[0]):
            row = attn[t, a, :row_len[t]].astype(np.float64)
            top = np.argsort(-row, kind="stable")[:K]
            c = int(((top >= span[t, 0]) & (top <= span[t, 1])).sum())
            # brute force: token j is in the top K iff fewer than K tokens beat it (larger value, or equal and earlier)
            beats = [(int((row > row[j]).sum()) + int((row[:j] == row[j]).sum())) for j in range(span[t, 0], span[t, 1] + 1)]
            assert c == sum(b < K for b in beats)
            tot += c
            mean += c / K
        assert counts[a] == tot and np.isclose(s[a], mean / attn.shape[0], rtol=0, atol=1e-15)


def test_closed_forms():
    T, H, L, K = 3, 2, 100, 24
    attn = np.zeros((T, H, L))
    attn[:, 0] = np.linspace(1.0, 0.0, L)            # strictly decreasing: the top K are tokens 0 .. K-1
    attn[:, 1] = np.linspace(0.0, 1.0, L)            # strictly increasing: tokens L-K .. L-1
    row_len = np.full(T, L, dtype=np.int32)
    span = np.array([[0, L - 1], [10, 29], [90, 99]], dtype=np.int32)
    s, counts = oracle.hit_score(attn, row_len, span, K)
    assert list(counts) == [24 + 14 + 0, 24 + 0 + 10]
    assert np.allclose(s, [(1 + 14 / 24 + 0) / 3, (1 + 0 + 10 / 24) / 3])
    # ties go to the lower token index; a row shorter than K contributes all of its tokens
    flat = np.ones((1, 1, 50))
    s, c = oracle.hit_score(flat, np.array([50]), np.array([[20, 30]]), K)
    assert c[0] == 4 and np.isclose(s[0], 4 / 24)     # top 24 = tokens 0..23, of which 20..23 lie in the span
    s, c = oracle.hit_score(flat, np.array([10]), np.array([[5, 30]]), K)
    assert c[0] == 5 and np.isclose(s[0], 5 / 24)
    # grounded heads score higher on the synthetic rows, and the score is a ratio
    attn, row_len, span, g = wl.attention_rows(n_steps=20, n_heads=16, n_audio=400, seed=1)
    s, _ = oracle.hit_score(attn, row_len, span, K)
    assert (s >= 0).all() and (s <= 1).all() and s[np.argmax(g)] > s[np.argmin(g)]
