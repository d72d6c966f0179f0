"""Thin ctypes binding over libaudiokv.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point it calls (see
include/audiokv.h); tensors are torch CUDA tensors whose data pointers are handed over as
they are, and the stream is torch's current stream. There is no fallback: if the CUDA
library cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaudiokv.so")

AUDIOKV_F32, AUDIOKV_BF16 = 0, 1
(AUDIOKV_SMOOTH_SSS, AUDIOKV_SMOOTH_FIXED_FRACTION, AUDIOKV_SMOOTH_ENERGY_NO_MEAN, AUDIOKV_SMOOTH_AVG_POOL,
 AUDIOKV_SMOOTH_MAX_POOL) = range(5)
AUDIOKV_OK, AUDIOKV_EINVAL, AUDIOKV_EALIGN, AUDIOKV_EUNSUPPORTED = 0, -1, -2, -3
AUDIOKV_EWORKSPACE, AUDIOKV_ECUDA, AUDIOKV_ETIMEOUT, AUDIOKV_EDEVICE = -4, -5, -6, -7


class AudioKVError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = f"{where}: {lib().audiokv_strerror(status).decode()} ({status})"
        super().__init__(msg + (f": {detail}" if detail else ""))


class audiokv_params(ctypes.Structure):
    _fields_ = [
        ("dtype", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("n_req", ctypes.c_int32),
        ("seq_len", ctypes.POINTER(ctypes.c_int32)), ("window", ctypes.c_int32),
        ("q_stride_req", ctypes.c_int64), ("q_stride_layer", ctypes.c_int64), ("q_stride_tok", ctypes.c_int64),
        ("q_stride_head", ctypes.c_int64),
        ("kv_stride_layer", ctypes.c_int64), ("kv_stride_tok", ctypes.c_int64), ("kv_stride_head", ctypes.c_int64),
        ("kv_req_offset", ctypes.POINTER(ctypes.c_int64)),
        ("softmax_scale", ctypes.c_float), ("rho", ctypes.c_float), ("alpha", ctypes.c_float),
        ("transition_bins", ctypes.c_int32), ("base_per_head", ctypes.c_int32),
        ("smooth_mode", ctypes.c_int32), ("smooth_kappa", ctypes.c_float), ("pool_kernel", ctypes.c_int32),
        ("q_req_offset", ctypes.POINTER(ctypes.c_int64)),
        ("page_size", ctypes.c_int32), ("n_pages", ctypes.c_int32), ("page_table", ctypes.c_void_p),
        ("page_table_stride", ctypes.c_int64),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C library. Raises if it has not been built (run paper_2604_06694_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_06694_b200.build`; "
                               "there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        pp = ctypes.POINTER(audiokv_params)
        L.audiokv_params_size.restype = sz
        L.audiokv_params_size.argtypes = []
        if L.audiokv_params_size() != ctypes.sizeof(audiokv_params):
            raise RuntimeError(f"audiokv_params is {L.audiokv_params_size()} bytes in {LIB_PATH} and "
                               f"{ctypes.sizeof(audiokv_params)} in this binding: rebuild the library")
        L.audiokv_strerror.restype = ctypes.c_char_p
        L.audiokv_strerror.argtypes = [ctypes.c_int]
        L.audiokv_budget_from_ratio.restype = i64
        L.audiokv_budget_from_ratio.argtypes = [ctypes.c_double, i32, i32, i32]
        L.audiokv_scores_len.restype = i64
        L.audiokv_scores_len.argtypes = [pp]
        L.audiokv_workspace_bytes.restype = sz
        L.audiokv_workspace_bytes.argtypes = [pp]
        L.audiokv_workspace_bytes_host.restype = sz
        L.audiokv_workspace_bytes_host.argtypes = [pp, i64, i64, ctypes.POINTER(i64)]
        L.audiokv_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, sz]
        L.audiokv_destroy.argtypes = [vp]
        L.audiokv_last_device_status.argtypes = [vp, vp]
        L.audiokv_last_cuda_error.restype = ctypes.c_char_p
        L.audiokv_last_cuda_error.argtypes = [vp]
        L.audiokv_launch_count.restype = i64
        L.audiokv_launch_count.argtypes = [vp]
        L.audiokv_last_score_path.argtypes = [vp]
        L.audiokv_last_score_path.restype = ctypes.c_char_p
        L.audiokv_set_wait_limit.argtypes = [i64]
        L.audiokv_set_wait_limit.restype = i64
        L.audiokv_profile_enable.argtypes = [vp, ctypes.c_int]
        L.audiokv_profile_enable.restype = ctypes.c_int
        L.audiokv_profile_count.argtypes = [vp]
        L.audiokv_profile_count.restype = ctypes.c_int
        L.audiokv_profile_name.argtypes = [vp, ctypes.c_int]
        L.audiokv_profile_name.restype = ctypes.c_char_p
        L.audiokv_profile_ms.argtypes = [vp, ctypes.c_int]
        L.audiokv_profile_ms.restype = ctypes.c_float
        L.audiokv_score.argtypes = [vp, pp, vp, vp, vp, vp]
        L.audiokv_score_noalloc.argtypes = [ctypes.c_int, pp, vp, vp, vp, vp]
        L.audiokv_score_noalloc.restype = ctypes.c_int
        L.audiokv_smooth.argtypes = [vp, pp, vp, vp, vp, vp]
        L.audiokv_allocate.argtypes = [vp, pp, vp, ctypes.POINTER(i64), vp, vp, vp]
        L.audiokv_select_gather.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.audiokv_evict.argtypes = [vp, pp, vp, vp, vp, vp, ctypes.POINTER(i64), vp, vp, vp, vp, vp, vp]
        L.audiokv_evict_kstar.argtypes = [vp, vp, vp]
        L.audiokv_evict_kstar.restype = ctypes.c_int
        L.audiokv_evict_budgeted.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.audiokv_evict_budgeted.restype = ctypes.c_int
        L.audiokv_reevict_workspace_bytes.restype = sz
        L.audiokv_reevict_workspace_bytes.argtypes = [pp, ctypes.POINTER(i32)]
        L.audiokv_reevict.argtypes = [vp, pp, vp, vp, vp, ctypes.POINTER(i32), ctypes.POINTER(i32), vp, vp, vp, vp, vp]
        L.audiokv_reevict.restype = ctypes.c_int
        L.audiokv_selection_spread.argtypes = [vp, pp, vp, vp, i32, vp, vp, vp]
        L.audiokv_selection_spread.restype = ctypes.c_int
        L.audiokv_hit_score.argtypes = [vp, vp, i32, i32, i64, vp, vp, i32, vp, vp, vp]
        L.audiokv_hit_score.restype = ctypes.c_int
        L.audiokv_evict_host.argtypes = [vp, pp, vp, i64, vp, vp, i64, vp, ctypes.POINTER(i64), vp, vp, vp, vp, vp, vp]
        for n in ("audiokv_create", "audiokv_destroy", "audiokv_last_device_status", "audiokv_score",
                  "audiokv_smooth", "audiokv_allocate", "audiokv_select_gather", "audiokv_evict",
                  "audiokv_evict_host"):
            getattr(L, n).restype = ctypes.c_int
        _lib = L
    return _lib


class Problem:
    """Owns an audiokv_params struct and the host arrays it points to."""

    def __init__(self, dtype: int, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 seq_lens: Sequence[int], window: int, q_strides: Sequence[int], kv_strides: Sequence[int],
                 kv_req_offset: Optional[Sequence[int]] = None, softmax_scale: float = 0.0, rho: float = 0.5,
                 alpha: float = 0.5, transition_bins: int = 4, base_per_head: int = 0, smooth_mode: int = 0,
                 smooth_kappa: float = 0.0, pool_kernel: int = 1, q_req_offset: Optional[Sequence[int]] = None,
                 page_size: int = 0, n_pages: int = 0, page_table: Optional[torch.Tensor] = None):
        n = len(seq_lens)
        self._qoff = (ctypes.c_int64 * n)(*[int(x) for x in q_req_offset]) if q_req_offset is not None else None
        self._seq = (ctypes.c_int32 * n)(*[int(x) for x in seq_lens])
        self._off = (ctypes.c_int64 * n)(*[int(x) for x in kv_req_offset]) if kv_req_offset is not None else None
        p = audiokv_params()
        p.dtype, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim = dtype, n_layers, n_q_heads, n_kv_heads, head_dim
        p.n_req, p.window = n, window
        p.seq_len = ctypes.cast(self._seq, ctypes.POINTER(ctypes.c_int32))
        p.q_stride_req, p.q_stride_layer, p.q_stride_tok, p.q_stride_head = [int(x) for x in q_strides]
        p.kv_stride_layer, p.kv_stride_tok, p.kv_stride_head = [int(x) for x in kv_strides]
        p.kv_req_offset = ctypes.cast(self._off, ctypes.POINTER(ctypes.c_int64)) if self._off is not None else None
        p.softmax_scale, p.rho, p.alpha = softmax_scale, rho, alpha
        p.transition_bins, p.base_per_head = transition_bins, base_per_head
        p.smooth_mode, p.smooth_kappa, p.pool_kernel = smooth_mode, smooth_kappa, pool_kernel
        p.q_req_offset = ctypes.cast(self._qoff, ctypes.POINTER(ctypes.c_int64)) if self._qoff is not None else None
        if page_size:
            # page_table: CUDA int32 [n_req][stride], kept alive here; the kv strides then describe the pool
            if page_table is None or not page_table.is_cuda or page_table.dtype != torch.int32 or page_table.dim() != 2 \
                    or not page_table.is_contiguous():
                raise ValueError("page_table must be a contiguous CUDA int32 tensor [n_req][stride]")
            self._page_table = page_table
            p.page_size, p.n_pages = page_size, n_pages
            p.page_table, p.page_table_stride = page_table.data_ptr(), page_table.shape[1]
        self.p = p
        self.seq_lens = [int(x) for x in seq_lens]

    @property
    def ref(self):
        return ctypes.byref(self.p)

    @property
    def total_heads(self) -> int:
        return self.p.n_req * self.p.n_layers * self.p.n_kv_heads

    @classmethod
    def from_workload(cls, w, **over) -> "Problem":
        """Problem for a paper_2604_06694_b200.workloads.Workload (layouts as documented there)."""
        s = w.spec
        kvs = w.kv_strides()
        kw = dict(dtype=AUDIOKV_F32 if s.dtype == "f32" else AUDIOKV_BF16, n_layers=s.n_layers,
                  n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, seq_lens=s.seq_lens,
                  window=s.window, q_strides=w.q_strides(), kv_strides=kvs,
                  kv_req_offset=[int(c) * kvs[1] for c in w.cu_seqlen[:-1]], rho=s.rho, alpha=s.alpha,
                  transition_bins=s.transition_bins, base_per_head=w.base)
        kw.update(over)
        return cls(**kw)


def audiokv_strerror(status: int) -> str:
    return lib().audiokv_strerror(status).decode()


def audiokv_budget_from_ratio(c: float, n_heads_total: int, seq_len: int, window: int) -> int:
    return int(lib().audiokv_budget_from_ratio(c, n_heads_total, seq_len, window))


def audiokv_set_wait_limit(cycles: int) -> int:
    """Limit (SM clock cycles) of the waits inside the scoring kernels; <= 0 restores the default. Returns the old one."""
    return int(lib().audiokv_set_wait_limit(int(cycles)))


def audiokv_scores_len(prob: Problem) -> int:
    return int(lib().audiokv_scores_len(prob.ref))


def audiokv_workspace_bytes(prob: Problem) -> int:
    return int(lib().audiokv_workspace_bytes(prob.ref))


def audiokv_workspace_bytes_host(prob: Problem, q_elems: int, kv_elems: int, total_budget: Sequence[int]) -> int:
    tb = (ctypes.c_int64 * len(total_budget))(*[int(x) for x in total_budget])
    return int(lib().audiokv_workspace_bytes_host(prob.ref, q_elems, kv_elems, tb))


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, name: str) -> ctypes.c_void_p:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


class Context:
    """audiokv_create / audiokv_destroy. `workspace_bytes` defaults to what `prob` needs."""

    def __init__(self, prob: Problem, device: int = 0, workspace_bytes: Optional[int] = None):
        if workspace_bytes is None:
            workspace_bytes = audiokv_workspace_bytes(prob)
            if workspace_bytes == 0:
                raise AudioKVError(AUDIOKV_EINVAL, "audiokv_workspace_bytes")
        h = ctypes.c_void_p()
        rc = lib().audiokv_create(ctypes.byref(h), device, workspace_bytes)
        if rc != 0:
            raise AudioKVError(rc, "audiokv_create")
        self.h = h
        self.workspace_bytes = workspace_bytes

    def close(self):
        if getattr(self, "h", None):
            lib().audiokv_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != 0:
            raise AudioKVError(rc, where, lib().audiokv_last_cuda_error(self.h).decode() if rc == AUDIOKV_ECUDA else "")

    def launch_count(self) -> int:
        return int(lib().audiokv_launch_count(self.h))

    def profile_enable(self, on: bool) -> None:
        self._check(lib().audiokv_profile_enable(self.h, int(on)), "audiokv_profile_enable")

    def profile_read(self):
        """[(kernel name, milliseconds)] of the last audiokv_evict call made while profiling was on."""
        n = lib().audiokv_profile_count(self.h)
        return [(lib().audiokv_profile_name(self.h, i).decode(), float(lib().audiokv_profile_ms(self.h, i)))
                for i in range(n)]

    def last_score_path(self) -> str:
        """"tcgen05", "fma" or "none": the kernels the last scoring on this context ran on."""
        return lib().audiokv_last_score_path(self.h).decode()

    def last_device_status(self) -> int:
        return int(lib().audiokv_last_device_status(self.h, _stream()))


def audiokv_score(ctx: Context, prob: Problem, q_win: torch.Tensor, k: torch.Tensor, scores: torch.Tensor) -> None:
    ctx._check(lib().audiokv_score(ctx.h, prob.ref, _dev(q_win, "q_win"), _dev(k, "k"), _dev(scores, "scores"),
                                   _stream()), "audiokv_score")


def audiokv_score_noalloc(prob: Problem, q_win: torch.Tensor, k: torch.Tensor, scores: torch.Tensor,
                          device: Optional[int] = None) -> None:
    """audiokv_score for callers that may not allocate device memory: no context, the scratch is a fixed
    8 MiB array inside the library (shared by all calls on the GPU, so keep calls ordered on one stream).
    Raises AudioKVError(AUDIOKV_EWORKSPACE) when the problem needs more scratch than that."""
    dev = q_win.device.index if device is None else device
    rc = lib().audiokv_score_noalloc(dev, prob.ref, _dev(q_win, "q_win"), _dev(k, "k"), _dev(scores, "scores"),
                                     _stream())
    if rc != 0:
        raise AudioKVError(rc, "audiokv_score_noalloc")


def audiokv_smooth(ctx: Context, prob: Problem, scores: torch.Tensor, smoothed: torch.Tensor,
                   kstar: Optional[torch.Tensor] = None) -> None:
    ks = _dev(kstar, "kstar") if kstar is not None else None
    ctx._check(lib().audiokv_smooth(ctx.h, prob.ref, _dev(scores, "scores"), _dev(smoothed, "smoothed"), ks,
                                    _stream()), "audiokv_smooth")


def _budget_array(total_budget: Sequence[int]):
    return (ctypes.c_int64 * len(total_budget))(*[int(x) for x in total_budget])


def audiokv_allocate(ctx: Context, prob: Problem, head_scores: torch.Tensor, total_budget: Sequence[int],
                     budgets: torch.Tensor, cu_kept: torch.Tensor) -> None:
    ctx._check(lib().audiokv_allocate(ctx.h, prob.ref, _dev(head_scores, "head_scores"), _budget_array(total_budget),
                                      _dev(budgets, "budgets"), _dev(cu_kept, "cu_kept"), _stream()),
               "audiokv_allocate")


def audiokv_select_gather(ctx: Context, prob: Problem, smoothed, budgets, cu_kept, k, v, k_out, v_out, kept_idx) -> None:
    ctx._check(lib().audiokv_select_gather(ctx.h, prob.ref, _dev(smoothed, "smoothed"), _dev(budgets, "budgets"),
                                           _dev(cu_kept, "cu_kept"), _dev(k, "k"), _dev(v, "v"), _dev(k_out, "k_out"),
                                           _dev(v_out, "v_out"), _dev(kept_idx, "kept_idx"), _stream()),
               "audiokv_select_gather")


def audiokv_evict(ctx: Context, prob: Problem, q_win, k, v, head_scores, total_budget: Sequence[int], k_out, v_out,
                  kept_idx, budgets, cu_kept) -> None:
    ctx._check(lib().audiokv_evict(ctx.h, prob.ref, _dev(q_win, "q_win"), _dev(k, "k"), _dev(v, "v"),
                                   _dev(head_scores, "head_scores"), _budget_array(total_budget), _dev(k_out, "k_out"),
                                   _dev(v_out, "v_out"), _dev(kept_idx, "kept_idx"), _dev(budgets, "budgets"),
                                   _dev(cu_kept, "cu_kept"), _stream()), "audiokv_evict")


def audiokv_evict_kstar(ctx: Context, kstar: torch.Tensor) -> None:
    """kstar: CUDA int32 [total heads], receives the cut-offs of the context's last pass."""
    ctx._check(lib().audiokv_evict_kstar(ctx.h, _dev(kstar, "kstar"), _stream()), "audiokv_evict_kstar")


def audiokv_evict_budgeted(ctx: Context, prob: Problem, q_win, k, v, budgets, k_out, v_out, kept_idx, cu_kept) -> None:
    """budgets: CUDA int32 [total heads], chosen by the caller (e.g. a slice of audiokv_allocate's output)."""
    ctx._check(lib().audiokv_evict_budgeted(ctx.h, prob.ref, _dev(q_win, "q_win"), _dev(k, "k"), _dev(v, "v"),
                                            _dev(budgets, "budgets"), _dev(k_out, "k_out"), _dev(v_out, "v_out"),
                                            _dev(kept_idx, "kept_idx"), _dev(cu_kept, "cu_kept"), _stream()),
               "audiokv_evict_budgeted")


def _i32_array(a: Sequence[int]):
    return (ctypes.c_int32 * len(a))(*[int(x) for x in a])


def audiokv_reevict_workspace_bytes(prob: Problem, cu_cache: Sequence[int]) -> int:
    return int(lib().audiokv_reevict_workspace_bytes(prob.ref, _i32_array(cu_cache)))


def audiokv_reevict(ctx: Context, prob: Problem, q_win, k_cache, v_cache, cu_cache: Sequence[int],
                    new_budgets: Sequence[int], k_out, v_out, kept_idx, cu_kept) -> None:
    """cu_cache and new_budgets are host sequences; everything else is a CUDA tensor."""
    ctx._check(lib().audiokv_reevict(ctx.h, prob.ref, _dev(q_win, "q_win"), _dev(k_cache, "k_cache"),
                                     _dev(v_cache, "v_cache"), _i32_array(cu_cache), _i32_array(new_budgets),
                                     _dev(k_out, "k_out"), _dev(v_out, "v_out"), _dev(kept_idx, "kept_idx"),
                                     _dev(cu_kept, "cu_kept"), _stream()), "audiokv_reevict")


def audiokv_selection_spread(ctx: Context, prob: Problem, kept_idx, cu_kept, n_bins: int, hist, stats) -> None:
    """hist: CUDA int32 [n_req][n_bins]; stats: CUDA fp32 [n_req][2] (balance, peak)."""
    ctx._check(lib().audiokv_selection_spread(ctx.h, prob.ref, _dev(kept_idx, "kept_idx"), _dev(cu_kept, "cu_kept"),
                                              n_bins, _dev(hist, "hist"), _dev(stats, "stats"), _stream()),
               "audiokv_selection_spread")


def audiokv_hit_score(ctx: Context, attn: torch.Tensor, row_len: torch.Tensor, span: torch.Tensor, top_k: int,
                      hit_counts: torch.Tensor, s_hit: torch.Tensor) -> None:
    """attn: CUDA fp32 [n_steps][n_heads][row_stride] (contiguous); row_len int32 [n_steps]; span int32 [n_steps][2]."""
    n_steps, n_heads, stride = attn.shape
    ctx._check(lib().audiokv_hit_score(ctx.h, _dev(attn, "attn"), n_steps, n_heads, stride, _dev(row_len, "row_len"),
                                       _dev(span, "span"), top_k, _dev(hit_counts, "hit_counts"), _dev(s_hit, "s_hit"),
                                       _stream()), "audiokv_hit_score")


def _host(t: torch.Tensor, name: str) -> ctypes.c_void_p:
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CPU tensor")
    return ctypes.c_void_p(t.data_ptr())


def audiokv_evict_host(ctx: Context, prob: Problem, q_win, k, v, head_scores, total_budget: Sequence[int], k_out,
                       v_out, kept_idx, budgets, cu_kept) -> None:
    """All tensors on the CPU (pinned for speed); the library copies in, evicts, copies out and waits."""
    ctx._check(lib().audiokv_evict_host(ctx.h, prob.ref, _host(q_win, "q_win"), q_win.numel(), _host(k, "k"),
                                        _host(v, "v"), k.numel(), _host(head_scores, "head_scores"),
                                        _budget_array(total_budget), _host(k_out, "k_out"), _host(v_out, "v_out"),
                                        _host(kept_idx, "kept_idx"), _host(budgets, "budgets"),
                                        _host(cu_kept, "cu_kept"), _stream()), "audiokv_evict_host")


lib()  # load now: a missing or broken CUDA library is an import error, never a silent fallback
