"""Seeded synthetic workloads for the AudioKV eviction pass.

This module only draws inputs. It holds none of the method's arithmetic and is
the one piece of code that both the CUDA parity tests and the CPU oracle's tests
use, so that the two sides see identical bytes.

The paper evaluates on speech corpora with Qwen2.5-Omni, Qwen3-Omni and Gemma-3n
checkpoints. Neither is available offline, so the inputs here reproduce the
shapes of those models' attention stacks and the structure the paper argues from:
audio tokens vary slowly along time (an AR(1) process along the token axis), text
tokens are independent, the first tokens may be attention sinks with a large key
norm, and only a few heads are strongly audio-critical (Beta(0.5, 2) scores).

Layouts (elements, last dimension contiguous):
  K, V : [n_layers][n_kv_heads][sum_L][head_dim]  -- requests concatenated along tokens
  Q    : [n_req][n_layers][W][n_q_heads][head_dim] -- the last W query rows of each request
  S    : [n_req][n_layers][n_kv_heads] float32     -- audio-criticality score per KV head
"""
from __future__ import annotations

import dataclasses
import math
import os
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch
from scipy.signal import lfilter


@dataclasses.dataclass
class WorkloadSpec:
    name: str
    dtype: str                    # "f32" | "bf16"
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_lens: List[int]           # one entry per request
    audio_frac: List[float]       # fraction of each request's tokens that are audio
    n_sink: int                   # leading tokens whose K rows are scaled by 8
    window: int = 32
    keep: float = 0.4
    ar_rho: float = 0.95
    ar_rho_range: Optional[Sequence[float]] = None   # per-(layer, head) rho ~ U(lo, hi) when set
    head_score_dist: str = "beta"  # "beta" -> Beta(0.5, 2); "uniform" -> U(0, 1)
    rho: float = 0.5              # SSS cut-off ratio
    alpha: float = 0.5            # SSS mixing coefficient
    transition_bins: int = 4      # SSS cosine band width T


def config(i: int, seed: int = 0) -> WorkloadSpec:
    """The five benchmark configurations, smallest first; index 1 is the one the benchmark line is quoted on."""
    if i == 0:
        return WorkloadSpec("c1_tiny_f32", "f32", 1, 8, 2, 64, [1024], [768 / 1024], 1, head_score_dist="uniform")
    if i == 1:
        return WorkloadSpec("c2_qwen25omni7b_L8k", "bf16", 28, 28, 4, 128, [8192], [7500 / 8192], 0)
    if i == 2:
        return WorkloadSpec("c3_qwen25omni7b_L32k", "bf16", 28, 28, 4, 128, [32768], [0.9], 0,
                            ar_rho_range=(0.85, 0.99))
    if i == 3:
        return WorkloadSpec("c4_qwen3omni30b_L16k", "bf16", 48, 32, 4, 128, [16384], [0.85], 4)
    if i == 4:
        rng = np.random.Generator(np.random.Philox(key=[seed, 0xC5]))
        lens = [int(math.floor(math.exp(rng.uniform(math.log(2048), math.log(32768))))) for _ in range(8)]
        fr = [float(rng.uniform(0.80, 0.95)) for _ in range(8)]
        return WorkloadSpec("c5_gemma3n_e4b_ragged8", "bf16", 35, 8, 2, 256, lens, fr, 0)
    raise ValueError(i)


def kept_total(spec: WorkloadSpec, L: int) -> int:
    """Total rows one request keeps over all heads at the spec's retention ratio: floor(c * N * L)."""
    n = spec.n_layers * spec.n_kv_heads
    return int(math.floor(spec.keep * n * L))


def base_per_head(spec: WorkloadSpec, L: int) -> int:
    """Uniform base allocation r used by the benchmark workloads: a tenth of a uniform head's non-window share."""
    return max(0, int(math.floor(0.1 * (math.floor(spec.keep * L) - spec.window))))


@dataclasses.dataclass
class Workload:
    spec: WorkloadSpec
    q: np.ndarray                 # raw storage: float32, or uint16 holding bf16 bits
    k: np.ndarray
    v: np.ndarray
    head_scores: np.ndarray       # float32 [n_req][n_layers][n_kv_heads]
    cu_seqlen: np.ndarray         # int64 [n_req + 1] token offsets of the requests
    total_budget: np.ndarray      # int64 [n_req]
    base: int                     # r (tokens per head)
    layer_begin: int = 0          # a layer shard: spec.n_layers layers starting here; head_scores and
    full_layers: Optional[int] = None  # total_budget still cover the full_layers layers of the whole stack

    @property
    def n_req(self) -> int:
        return len(self.spec.seq_lens)

    @property
    def sum_L(self) -> int:
        return int(self.cu_seqlen[-1])

    def kv_strides(self):
        """(layer, token, head) strides of K and V in elements."""
        s = self.spec
        return (s.n_kv_heads * self.sum_L * s.head_dim, s.head_dim, self.sum_L * s.head_dim)

    def q_strides(self):
        """(request, layer, token, head) strides of Q in elements."""
        s = self.spec
        per_tok = s.n_q_heads * s.head_dim
        return (s.n_layers * s.window * per_tok, s.window * per_tok, per_tok, s.head_dim)

    def torch_dtype(self):
        return torch.float32 if self.spec.dtype == "f32" else torch.bfloat16

    def as_torch(self, a: np.ndarray) -> torch.Tensor:
        t = torch.from_numpy(a)
        return t if self.spec.dtype == "f32" or a.dtype != np.uint16 else t.view(torch.bfloat16)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round once (nearest even) to the storage type; bf16 is returned as its uint16 bit pattern."""
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.uint16).numpy()


def _ar1_inplace(x: np.ndarray, rho: float) -> None:
    """x[t] <- rho x[t-1] + sqrt(1 - rho^2) x[t] along axis 0, x[0] kept: stationary, unit variance."""
    if x.shape[0] < 2:
        return
    g = math.sqrt(1.0 - rho * rho)
    drive = x * g
    drive[0] = x[0]
    x[...] = lfilter([1.0], [1.0, -rho], drive, axis=0)


def generate(spec: WorkloadSpec, seed: int = 0, layers: Optional[int] = None,
             layer_range: Optional[Tuple[int, int]] = None, workers: Optional[int] = None) -> Workload:
    """Draw one workload. `layers` truncates the stack (the first `layers` layers) for small parity cases;
    budgets are then computed for the truncated stack. `layer_range` = (l0, l1) draws only layers l0..l1-1 of
    that stack, bit-identical to the same layers of the full draw (a layer shard of a multi-GPU run): q, k, v hold
    l1 - l0 layers, while head_scores and total_budget stay those of the whole stack, which the allocation needs.
    `workers`: threads drawing (request, layer) pairs side by side (the result does not depend on it)."""
    if layers is not None:
        spec = dataclasses.replace(spec, n_layers=int(layers))
    NL, Hq, Hkv, d, W = spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.window
    l0, l1 = (0, NL) if layer_range is None else (int(layer_range[0]), int(layer_range[1]))
    if not 0 <= l0 < l1 <= NL:
        raise ValueError("layer_range outside the stack")
    lens = list(spec.seq_lens)
    cu = np.zeros(len(lens) + 1, dtype=np.int64)
    cu[1:] = np.cumsum(lens)
    sumL = int(cu[-1])
    G = Hq // Hkv
    st = np.uint16 if spec.dtype == "bf16" else np.float32
    k = np.zeros((l1 - l0, Hkv, sumL, d), dtype=st)
    v = np.zeros((l1 - l0, Hkv, sumL, d), dtype=st)
    q = np.zeros((len(lens), l1 - l0, W, Hq, d), dtype=st)
    S = np.zeros((len(lens), NL, Hkv), dtype=np.float32)
    def draw_layer(r: int, l: int) -> None:
        # every (request, layer) has a generator of its own, so the draw does not depend on the order of the calls
        L = lens[r]
        n_audio = int(round(spec.audio_frac[r] * L))
        rng = np.random.Generator(np.random.Philox(key=[seed, (r << 20) + l + 1]))
        for h in range(Hkv):
            rho = spec.ar_rho if spec.ar_rho_range is None else float(rng.uniform(*spec.ar_rho_range))
            for dst, is_k in ((k, True), (v, False)):
                x = rng.standard_normal(size=(L, d), dtype=np.float32)
                _ar1_inplace(x[:n_audio], rho)
                if is_k and spec.n_sink:
                    x[: spec.n_sink] *= 8.0
                dst[l - l0, h, cu[r]:cu[r] + L] = _store(x, spec.dtype)
            # window queries of this KV head's group; window tokens inside the audio segment continue an AR(1) chain
            xq = rng.standard_normal(size=(W, G * d), dtype=np.float32)
            n_aw = max(0, min(W, n_audio - (L - W)))
            _ar1_inplace(xq[:n_aw], rho)
            q[r, l - l0, :, h * G:(h + 1) * G, :] = _store(xq, spec.dtype).reshape(W, G, d)

    for r, L in enumerate(lens):
        rng_s = np.random.Generator(np.random.Philox(key=[seed, 1000 + r]))
        if spec.head_score_dist == "uniform":
            S[r] = rng_s.uniform(0.0, 1.0, size=(NL, Hkv)).astype(np.float32)
        else:
            S[r] = rng_s.beta(0.5, 2.0, size=(NL, Hkv)).astype(np.float32)
    jobs = [(r, l) for r in range(len(lens)) for l in range(l0, l1)]
    n_workers = min(len(jobs), workers if workers is not None else min(16, os.cpu_count() or 1))
    if n_workers > 1:
        with ThreadPoolExecutor(n_workers) as pool:
            list(pool.map(lambda rl: draw_layer(*rl), jobs))
    else:
        for rl in jobs:
            draw_layer(*rl)
    B = np.array([kept_total(spec, L) for L in lens], dtype=np.int64)
    base = base_per_head(spec, min(lens))
    if layer_range is None:
        return Workload(spec, q, k, v, S, cu, B, base)
    return Workload(dataclasses.replace(spec, n_layers=l1 - l0), q, k, v, S, cu, B, base, layer_begin=l0, full_layers=NL)


def layer_shard(n_layers: int, world: int, rank: int) -> Tuple[int, int]:
    """Layers [l0, l1) of rank `rank` when the stack is dealt out in contiguous runs, the first n_layers % world ranks
    taking one more."""
    q, rem = divmod(n_layers, world)
    l0 = rank * q + min(rank, rem)
    return l0, l0 + q + (1 if rank < rem else 0)


def shard_heads(n_req: int, n_layers: int, n_kv_heads: int, l0: int, l1: int) -> np.ndarray:
    """Flat indices u = (r * n_layers + l) * n_kv_heads + h of the heads of layers l0..l1-1, in the order the shard's
    own flat index runs (request, layer, head)."""
    r, l, h = np.meshgrid(np.arange(n_req), np.arange(l0, l1), np.arange(n_kv_heads), indexing="ij")
    return ((r * n_layers + l) * n_kv_heads + h).reshape(-1)


def attention_rows(n_steps: int, n_heads: int, n_audio: int, n_text0: int = 16, seed: int = 0, word_tokens: int = 12):
    """Synthetic decode-step attention rows for the offline head-score statistic (the paper records them with hooks
    on a real model): step t attends over L_t = n_audio + n_text0 + t tokens; the word generated at step t spans
    `word_tokens` audio tokens that advance with t (speech is read left to right); head a puts a share g_a of its
    logit mass on that span (g ~ Beta(0.5, 2): few strongly audio-grounded heads) on top of i.i.d. noise and a sink
    at token 0. Returns (attn float32 [n_steps][n_heads][Lmax] zero-padded, row_len int32, span int32 [n_steps][2],
    grounding float64 [n_heads])."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0xA77]))
    Lmax = n_audio + n_text0 + n_steps
    attn = np.zeros((n_steps, n_heads, Lmax), dtype=np.float32)
    row_len = np.array([n_audio + n_text0 + t for t in range(n_steps)], dtype=np.int32)
    span = np.zeros((n_steps, 2), dtype=np.int32)
    g = rng.beta(0.5, 2.0, size=n_heads)
    for t in range(n_steps):
        lo = min(n_audio - word_tokens, int(t * (n_audio - word_tokens) / max(1, n_steps - 1)))
        span[t] = (lo, lo + word_tokens - 1)
        L = int(row_len[t])
        z = rng.standard_normal(size=(n_heads, L))
        z[:, 0] += 4.0
        z[:, lo:lo + word_tokens] += 6.0 * g[:, None]
        z -= z.max(axis=1, keepdims=True)
        p = np.exp(z)
        attn[t, :, :L] = (p / p.sum(axis=1, keepdims=True)).astype(np.float32)
    return attn, row_len, span, g


@dataclasses.dataclass
class CompactedCache:
    """A cache that has been evicted once and has decoded `n_new` tokens since: per-head ragged rows."""
    spec: WorkloadSpec
    q: np.ndarray            # raw storage [n_req][n_layers][W][n_q_heads][d]: queries of the last W decoded tokens
    k: np.ndarray            # raw storage [rows][d], head u = (r * n_layers + l) * n_kv_heads + h at rows cu[u]..cu[u+1]
    v: np.ndarray
    cu: np.ndarray           # int32 [total heads + 1]
    new_budgets: np.ndarray  # int32 [total heads]: rows each head keeps after the re-eviction (window included)

    def q_strides(self):
        s = self.spec
        per_tok = s.n_q_heads * s.head_dim
        return (s.n_layers * s.window * per_tok, s.window * per_tok, per_tok, s.head_dim)

    def torch_dtype(self):
        return torch.float32 if self.spec.dtype == "f32" else torch.bfloat16

    def as_torch(self, a: np.ndarray) -> torch.Tensor:
        t = torch.from_numpy(a)
        return t if self.spec.dtype == "f32" or a.dtype != np.uint16 else t.view(torch.bfloat16)


def compacted_cache(spec: WorkloadSpec, n_new: int, seed: int = 0, layers: Optional[int] = None,
                    spread: float = 0.5) -> CompactedCache:
    """Each head of each request kept b_u rows at prefill, b_u drawn uniformly within +-spread of the request's
    mean budget (never below W + 1 nor above L), and has appended `n_new` decoded rows; the re-eviction brings it
    back to b_u. Kept rows are AR(1) like the audio keys of `generate`, decoded rows are white."""
    if layers is not None:
        spec = dataclasses.replace(spec, n_layers=int(layers))
    NL, Hq, Hkv, d, W = spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.window
    G = Hq // Hkv
    lens = list(spec.seq_lens)
    st = np.uint16 if spec.dtype == "bf16" else np.float32
    TH = len(lens) * NL * Hkv
    rng_b = np.random.Generator(np.random.Philox(key=[seed, 77]))
    cu = np.zeros(TH + 1, dtype=np.int64)
    budgets = np.zeros(TH, dtype=np.int32)
    u = 0
    for L in lens:
        mean = kept_total(spec, L) / (NL * Hkv)
        for _ in range(NL * Hkv):
            b = int(round(mean * (1.0 + spread * (2.0 * rng_b.random() - 1.0))))
            budgets[u] = min(max(b, W + 1), L)
            cu[u + 1] = cu[u] + budgets[u] + n_new
            u += 1
    rows = int(cu[-1])
    k = np.zeros((rows, d), dtype=st)
    v = np.zeros((rows, d), dtype=st)
    q = np.zeros((len(lens), NL, W, Hq, d), dtype=st)
    u = 0
    for r in range(len(lens)):
        for l in range(NL):
            rng = np.random.Generator(np.random.Philox(key=[seed, (r << 20) + l + 1 + (1 << 40)]))
            for h in range(Hkv):
                n_old = int(budgets[u])
                rho = spec.ar_rho if spec.ar_rho_range is None else float(rng.uniform(*spec.ar_rho_range))
                for dst, is_k in ((k, True), (v, False)):
                    x = rng.standard_normal(size=(n_old + n_new, d), dtype=np.float32)
                    _ar1_inplace(x[:n_old], rho)
                    if is_k and spec.n_sink:
                        x[: spec.n_sink] *= 8.0
                    dst[cu[u]:cu[u + 1]] = _store(x, spec.dtype)
                xq = rng.standard_normal(size=(W, G * d), dtype=np.float32)
                q[r, l, :, h * G:(h + 1) * G, :] = _store(xq, spec.dtype).reshape(W, G, d)
                u += 1
    return CompactedCache(spec, q, k, v, cu.astype(np.int32), budgets)


def paged_pool(w: Workload, page_size: int, seed: int = 0, spare: int = 3):
    """The K and V of `w` scattered into pools of pages, the way a serving stack's block allocator holds them.

    Returns (k_pool, v_pool, page_table, n_pages, kv_strides): pools are raw storage [n_layers][n_pages * page_size]
    [n_kv_heads][d] (token-major inside a page), page_table is int32 [n_req][max pages of a request] with -1 in unused
    slots, pages are handed out in a random order, `spare` pages belong to nobody, and every pool slot that holds no
    token (page tails, spare pages) is filled with NaN, which a correct reader never lets through.
    kv_strides = (layer, token, head) strides of the pools in elements."""
    s = w.spec
    NL, Hkv, d = s.n_layers, s.n_kv_heads, s.head_dim
    lens = list(s.seq_lens)
    per_req = [(L + page_size - 1) // page_size for L in lens]
    n_pages = sum(per_req) + spare
    rng = np.random.Generator(np.random.Philox(key=[seed, 4242]))
    order = rng.permutation(n_pages)
    table = np.full((len(lens), max(per_req)), -1, dtype=np.int32)
    nan = np.uint16(0x7FC0) if w.k.dtype == np.uint16 else np.float32(np.nan)
    k_pool = np.full((NL, n_pages * page_size, Hkv, d), nan, dtype=w.k.dtype)
    v_pool = np.full((NL, n_pages * page_size, Hkv, d), nan, dtype=w.v.dtype)
    nxt = 0
    for r, L in enumerate(lens):
        base = int(w.cu_seqlen[r])
        for i in range(per_req[r]):
            pg = int(order[nxt])
            nxt += 1
            table[r, i] = pg
            n = min(page_size, L - i * page_size)
            src = slice(base + i * page_size, base + i * page_size + n)
            dst = slice(pg * page_size, pg * page_size + n)
            k_pool[:, dst] = np.transpose(w.k[:, :, src], (0, 2, 1, 3))
            v_pool[:, dst] = np.transpose(w.v[:, :, src], (0, 2, 1, 3))
    strides = (n_pages * page_size * Hkv * d, Hkv * d, d)
    return k_pool, v_pool, table, n_pages, strides
