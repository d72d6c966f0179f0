"""Shared pieces of the GPU parity tests: run the oracle on a workload, compare with the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

import oracle

REL_TOL = 1e-3      # max relative error of scores / smoothed scores (fp32 accumulate from bf16 inputs)
KSTAR_TIE = 2e-5    # energy margin (relative to the total) below which an fp32 transform may move k* by one bin
# In the fused pass the transform's input is the GPU's own scores, which may differ from the oracle's by REL_TOL:
# a relative error e in the sequence moves every cumulative energy by up to 2 e of the total, so the cut-off may move
# whenever the oracle's margin is below that (plus the transform's own allowance).
FUSED_KSTAR_TIE = 2 * REL_TOL + KSTAR_TIE


def rel_err(g: np.ndarray, o: np.ndarray) -> float:
    """max_j |g_j - o_j| / max(|o_j|, mean_j |o_j|): smoothed scores cross zero, so small entries are
    measured against the head's mean magnitude."""
    o = np.asarray(o, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    if o.size == 0:
        return 0.0
    den = np.maximum(np.abs(o), np.abs(o).mean())
    den = np.where(den > 0, den, 1.0)
    return float(np.max(np.abs(g - o) / den))


def oracle_dtype(w) -> int:
    return oracle.F32 if w.spec.dtype == "f32" else oracle.BF16


def request_views(w, r):
    """(q_r, k, v, dims, q_strides(layer,tok,head), kv_strides, kv element offset) of request r for the oracle."""
    s = w.spec
    L = s.seq_lens[r]
    dims = (s.n_layers, s.window, s.n_q_heads, s.n_kv_heads, s.head_dim, L)
    off = int(w.cu_seqlen[r]) * w.kv_strides()[1]
    return w.q[r], w.k.reshape(-1)[off:], w.v.reshape(-1)[off:], dims, w.q_strides()[1:], w.kv_strides(), off


def oracle_scores(w, r, scale=None):
    s = w.spec
    q, k, _, dims, qs, kvs, _ = request_views(w, r)
    scale = scale if scale is not None else 1.0 / np.sqrt(s.head_dim)
    sc, wm = oracle.score(q, k, oracle_dtype(w), scale, qs, kvs, dims)
    return sc, wm


def check_kept(gpu_idx: np.ndarray, s_hat: np.ndarray, k: int, P: int, W: int, where: str):
    """gpu_idx: the GPU's kept indices of one head (ascending prefix part, then the window).
    s_hat: the ORACLE's smoothed scores. The sets must agree except among tokens whose score is
    within 1e-3 (relative) of the oracle's k-th value, and what the GPU kept must be valid."""
    assert len(gpu_idx) == k + W, where
    pre, win = gpu_idx[:k], gpu_idx[k:]
    assert np.array_equal(win, np.arange(P, P + W)), where
    if k:
        assert (np.diff(pre) > 0).all() and pre[0] >= 0 and pre[-1] < P, where
    want = oracle.select(s_hat, k)
    if np.array_equal(pre, want):
        return 0
    assert 0 < k < P, where
    theta = np.sort(s_hat)[::-1][k - 1]
    tol = REL_TOL * max(abs(theta), np.abs(s_hat).mean())
    diff = np.setxor1d(pre, want)
    assert (np.abs(s_hat[diff] - theta) <= tol).all(), f"{where}: kept sets differ away from the threshold"
    return len(diff)


def to_dev(w, a):
    return w.as_torch(a).cuda()
