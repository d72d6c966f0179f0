"""CPU oracle of the AudioKV eviction pass (ctypes wrapper over audiokv_oracle.cpp).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline call this; the CUDA library and its Python binding never import it.
The arithmetic lives in audiokv_oracle.cpp; this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "audiokv_oracle.cpp")
_LIB = os.path.join(_HERE, "libaudiokv_oracle.so")

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP over layers and heads). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.akvo_score.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, i32, i64, i64, i64, i64, i64, i64, f64, vp, vp]
        lib.akvo_rfft.argtypes = [vp, i32, i32, vp, vp]
        lib.akvo_irfft.argtypes = [vp, vp, i32, i32, vp]
        lib.akvo_sss.argtypes = [vp, i32, f64, f64, i32, i32, i32, vp, vp, vp, vp]
        lib.akvo_smooth_variant.argtypes = [vp, i32, i32, f64, f64, i32, i32, i32, vp, vp]
        lib.akvo_smooth_variant.restype = ctypes.c_int
        lib.akvo_hit_score.argtypes = [vp, i32, i32, ctypes.c_int64, vp, vp, i32, vp, vp]
        lib.akvo_hit_score.restype = ctypes.c_int
        lib.akvo_selection_spread.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        lib.akvo_selection_spread.restype = ctypes.c_int
        lib.akvo_allocate.argtypes = [vp, i32, i64, i32, i32, i32, vp]
        lib.akvo_select.argtypes = [vp, i32, i32, vp]
        lib.akvo_gather.argtypes = [vp, i32, i32, i64, vp, i32, vp]
        for name in ("akvo_score", "akvo_rfft", "akvo_irfft", "akvo_sss", "akvo_allocate", "akvo_select", "akvo_gather"):
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _check_raw(a: np.ndarray, dtype: int) -> np.ndarray:
    want = np.float32 if dtype == F32 else np.uint16
    if a.dtype != want:
        raise TypeError(f"expected {want} storage for dtype {dtype}, got {a.dtype}")
    return a


def score(q: np.ndarray, k: np.ndarray, dtype: int, scale: float, q_strides, k_strides, dims):
    """Observation-window scores of one request.

    q, k: raw storage (float32, or uint16 holding bf16 bits), any shape, addressed by
    strides in elements: q_strides = (layer, token, head), k_strides = (layer, token, head).
    dims = (n_layers, W, Hq, Hkv, d, L). Returns (s [NL, Hkv, P] float64, window_mass [NL, Hkv]).
    """
    NL, W, Hq, Hkv, d, L = dims
    _check_raw(q, dtype), _check_raw(k, dtype)
    P = L - W
    s = np.zeros((NL, Hkv, P), dtype=np.float64)
    wm = np.zeros((NL, Hkv), dtype=np.float64)
    rc = _load().akvo_score(_ptr(q), _ptr(k), dtype, NL, W, Hq, Hkv, d, L, *[int(x) for x in q_strides],
                            *[int(x) for x in k_strides], float(scale), _ptr(s), _ptr(wm))
    if rc != 0:
        raise ValueError(f"akvo_score rejected its arguments ({rc})")
    return s, wm


def rfft(x: np.ndarray, direct: bool = False):
    x = np.ascontiguousarray(x, dtype=np.float64)
    n = x.shape[0]
    re = np.zeros(n // 2 + 1)
    im = np.zeros(n // 2 + 1)
    rc = _load().akvo_rfft(_ptr(x), n, int(direct), _ptr(re), _ptr(im))
    if rc != 0:
        raise ValueError("akvo_rfft rejected its arguments")
    return re + 1j * im


def irfft(F: np.ndarray, n: int, direct: bool = False):
    re = np.ascontiguousarray(F.real, dtype=np.float64)
    im = np.ascontiguousarray(F.imag, dtype=np.float64)
    assert re.shape[0] == n // 2 + 1
    x = np.zeros(n)
    rc = _load().akvo_irfft(_ptr(re), _ptr(im), n, int(direct), _ptr(x))
    if rc != 0:
        raise ValueError("akvo_irfft rejected its arguments")
    return x


def sss(x: np.ndarray, rho: float, alpha: float, T: int, force_kstar: int = -1, direct: bool = False,
        want_energy: bool = False):
    """Spectral Score Smoothing of one score sequence. Returns (out, kstar, margin[, E])."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    n = x.shape[0]
    out = np.zeros(n)
    kstar = ctypes.c_int(0)
    margin = ctypes.c_double(0.0)
    E = np.zeros(n // 2 + 1) if want_energy else None
    rc = _load().akvo_sss(_ptr(x), n, float(rho), float(alpha), int(T), int(force_kstar), int(direct), _ptr(out),
                          ctypes.cast(ctypes.byref(kstar), ctypes.c_void_p),
                          ctypes.cast(ctypes.byref(margin), ctypes.c_void_p), _ptr(E) if want_energy else None)
    if rc != 0:
        raise ValueError("akvo_sss rejected its arguments")
    if want_energy:
        return out, kstar.value, margin.value, E
    return out, kstar.value, margin.value


FIXED_FRACTION, ENERGY_NO_MEAN, AVG_POOL, MAX_POOL = 1, 2, 3, 4


def smooth_variant(x: np.ndarray, mode: int, param: float, alpha: float, T: int = 0, pool: int = 1, direct: bool = False):
    """The smoothing variants for ablation-style runs (see akvo_smooth_variant). Returns (out, kstar)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    n = x.shape[0]
    out = np.zeros(n)
    kstar = ctypes.c_int(0)
    rc = _load().akvo_smooth_variant(_ptr(x), n, int(mode), float(param), float(alpha), int(T), int(pool), int(direct),
                                     _ptr(out), ctypes.cast(ctypes.byref(kstar), ctypes.c_void_p))
    if rc != 0:
        raise ValueError("akvo_smooth_variant rejected its arguments")
    return out, kstar.value


def hit_score(attn: np.ndarray, row_len: np.ndarray, span: np.ndarray, K: int = 24):
    """Offline head score: attn [n_steps][n_heads][row_stride], row_len [n_steps], span [n_steps][2] (inclusive).
    Returns (s_hit float64 [n_heads], counts int64 [n_heads])."""
    attn = np.ascontiguousarray(attn, dtype=np.float64)
    T, H, stride = attn.shape
    row_len = np.ascontiguousarray(row_len, dtype=np.int32)
    span = np.ascontiguousarray(span, dtype=np.int32).reshape(T, 2)
    counts = np.zeros(H, dtype=np.int64)
    s = np.zeros(H)
    rc = _load().akvo_hit_score(_ptr(attn), T, H, stride, _ptr(row_len), _ptr(span), int(K), _ptr(counts), _ptr(s))
    if rc != 0:
        raise ValueError("akvo_hit_score rejected its arguments")
    return s, counts


def selection_spread(kept: np.ndarray, cu_kept: np.ndarray, P: int, n_bins: int):
    """Histogram of one request's kept prefix tokens over n_bins stretches of the prefix, and its two summaries.
    kept: int32, the heads' indices back to back; cu_kept: int32 [N + 1], relative to kept[0].
    Returns (hist int64 [n_bins], balance, peak)."""
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    cu_kept = np.ascontiguousarray(cu_kept, dtype=np.int32)
    hist = np.zeros(n_bins, dtype=np.int64)
    bal, pk = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = _load().akvo_selection_spread(_ptr(kept), _ptr(cu_kept), len(cu_kept) - 1, int(P), int(n_bins), _ptr(hist),
                                       ctypes.byref(bal), ctypes.byref(pk))
    if rc != 0:
        raise ValueError("akvo_selection_spread rejected its arguments")
    return hist, bal.value, pk.value


def allocate(S: np.ndarray, B: int, w: int, r: int, L: int) -> np.ndarray:
    """Integer budgets of one request; S is the flat [layers*heads] float32 score table."""
    S = np.ascontiguousarray(S, dtype=np.float32).reshape(-1)
    b = np.zeros(S.shape[0], dtype=np.int32)
    rc = _load().akvo_allocate(_ptr(S), S.shape[0], int(B), int(w), int(r), int(L), _ptr(b))
    if rc != 0:
        raise ValueError(f"akvo_allocate rejected its arguments ({rc})")
    return b


def select(s_hat: np.ndarray, k: int) -> np.ndarray:
    s_hat = np.ascontiguousarray(s_hat, dtype=np.float64)
    idx = np.zeros(k, dtype=np.int32)
    rc = _load().akvo_select(_ptr(s_hat), s_hat.shape[0], int(k), _ptr(idx))
    if rc != 0:
        raise ValueError("akvo_select rejected its arguments")
    return idx


def gather(src: np.ndarray, dtype: int, d: int, stride_tok: int, idx: np.ndarray) -> np.ndarray:
    """Rows idx of one head's cache (raw storage, rows stride_tok elements apart) packed to [len(idx), d]."""
    _check_raw(src, dtype)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    dst = np.zeros((idx.shape[0], d), dtype=src.dtype)
    rc = _load().akvo_gather(_ptr(src), dtype, d, int(stride_tok), _ptr(idx), idx.shape[0], _ptr(dst))
    if rc != 0:
        raise ValueError("akvo_gather rejected its arguments")
    return dst


def evict_request(q, k, v, dtype, dims, q_strides, kv_strides, scale, head_scores, B, r, rho, alpha, T,
                  force_kstar=None):
    """The whole pass for one request, step by step in the paper's order.

    Returns dict(scores, smoothed, kstar, margin, budgets, kept (list per head), k_out, v_out (lists)).
    """
    NL, W, Hq, Hkv, d, L = dims
    P = L - W
    s, _ = score(q, k, dtype, scale, q_strides, kv_strides, dims)
    sm = np.zeros_like(s)
    ks = np.zeros((NL, Hkv), dtype=np.int32)
    mg = np.zeros((NL, Hkv))
    for l in range(NL):
        for h in range(Hkv):
            fk = -1 if force_kstar is None else int(force_kstar[l, h])
            sm[l, h], ks[l, h], mg[l, h] = sss(s[l, h], rho, alpha, T, force_kstar=fk)
    b = allocate(np.asarray(head_scores, dtype=np.float32).reshape(-1), B, W, r, L).reshape(NL, Hkv)
    kept, k_out, v_out = [], [], []
    kflat, vflat = k.reshape(-1), v.reshape(-1)
    for l in range(NL):
        for h in range(Hkv):
            idx = select(sm[l, h], int(b[l, h]) - W)
            idx = np.concatenate([idx, np.arange(P, L, dtype=np.int32)])
            kept.append(idx)
            base = l * kv_strides[0] + h * kv_strides[2]
            k_out.append(gather(kflat[base:], dtype, d, kv_strides[1], idx))
            v_out.append(gather(vflat[base:], dtype, d, kv_strides[1], idx))
    return dict(scores=s, smoothed=sm, kstar=ks, margin=mg, budgets=b, kept=kept, k_out=k_out, v_out=v_out)
