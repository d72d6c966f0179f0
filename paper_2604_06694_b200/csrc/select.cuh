// Top-k of one head's scores by radix select, for a block of kSelThreads threads.
// Shared by the stand-alone selection kernel and by the smoothing kernel, which selects
// straight from the smoothed scores it still holds on chip.
#pragma once

#include "common.cuh"

namespace akv {

constexpr int kSelThreads = 1024;

// Order-preserving map float -> uint32 (larger float, larger key); -0 and +0 share a key.
__device__ __forceinline__ uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelBins = 2048;  // 11-bit digits: three passes (11 + 11 + 10 bits) cover the 32-bit key

struct SelectSmem {
  int hist[kSelBins];
  int wsum[32];
  int weq[32];
  uint32_t prefix;
  int want;
};

__device__ __forceinline__ int block_excl_scan_int(int v, int* wsum, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) wsum[warp] = inc;
  __syncthreads();
  int ws = wsum[lane], winc = ws;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += t;
  }
  *total = __shfl_sync(0xffffffffu, winc, 31);
  return __shfl_sync(0xffffffffu, winc - ws, warp) + inc - v;
}

// Writes to `out` the k prefix tokens (of P) with the largest keys, ties to the lower index, in
// ascending token order, then the W window tokens P .. P+W-1. key_at(j) gives the key of token j.
// Every thread of the block calls this with the same arguments. Three radix passes (11, 11 and 10 bits) find
// the k-th largest key; the bin that holds it is located by a block-wide scan over the counts. The compaction
// gives every warp a contiguous stretch of tokens, 32 neighbours at a time: ballots rank the kept tokens inside
// the warp, one exchange of the warps' totals ranks the warps.
template <typename KeyAt>
__device__ __forceinline__ void select_topk(KeyAt key_at, int P, int W, int k, int32_t* __restrict__ out,
                                            SelectSmem* sm, int* __restrict__ status) {
  static_assert(kSelBins == 2 * kSelThreads, "every thread owns two bins of the histogram");
  uint32_t thr = 0;  // key of the k-th largest element
  int need_eq = 0;   // how many elements equal to thr are kept (those with the lowest indices)
  if (k > 0 && k < P) {
    // thread t owns bins 2047 - 2t and 2046 - 2t (descending): `above` counts the keys in higher bins
    const int b_hi = kSelBins - 1 - 2 * static_cast<int>(threadIdx.x), b_lo = b_hi - 1;
    __syncthreads();
    if (threadIdx.x == 0) {
      sm->prefix = 0u;
      sm->want = k;
    }
    sm->hist[b_hi] = 0;
    sm->hist[b_lo] = 0;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;
      const int bits = pass == 2 ? 10 : 11;
      const uint32_t dmask = (1u << bits) - 1u;
      __syncthreads();  // the histogram is clear; prefix and want of the pass before are set
      const uint32_t prefix = sm->prefix;
      const int want = sm->want;
      const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + bits));
      for (int j = threadIdx.x; j < P; j += kSelThreads) {
        const uint32_t key = key_at(j);
        if ((key & pmask) == prefix) atomicAdd(&sm->hist[(key >> shift) & dmask], 1);
      }
      __syncthreads();
      const int c_hi = sm->hist[b_hi], c_lo = sm->hist[b_lo];
      sm->hist[b_hi] = 0;  // its owner clears a bin for the next pass as soon as it has read it
      sm->hist[b_lo] = 0;
      int tot;
      const int above = block_excl_scan_int(c_hi + c_lo, sm->wsum, &tot);
      if (above < want && want <= above + c_hi) {
        sm->prefix = prefix | (static_cast<uint32_t>(b_hi) << shift);
        sm->want = want - above;
      } else if (above + c_hi < want && want <= above + c_hi + c_lo) {
        sm->prefix = prefix | (static_cast<uint32_t>(b_lo) << shift);
        sm->want = want - above - c_hi;
      }
    }
    __syncthreads();
    thr = sm->prefix;
    need_eq = sm->want;
  } else if (k == P) {
    thr = 0u;
    need_eq = P;  // every key is >= 0: keep all
  }

  // ordered compaction: warp w owns tokens [w * chunk, (w + 1) * chunk), lane l looks at token j0 + l of each row of 32
  constexpr int kWarps = kSelThreads / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t lt = (1u << lane) - 1u;
  const int chunk = ((P + kWarps - 1) / kWarps + 31) & ~31;
  const int c0 = min(P, warp * chunk), c1 = min(P, c0 + chunk);
  int n_gt = 0, n_eq = 0;
  if (k > 0) {
    for (int j0 = c0; j0 < c1; j0 += 32) {
      const int j = j0 + lane;
      const uint32_t key = j < c1 ? key_at(j) : 0u;
      n_gt += __popc(__ballot_sync(0xffffffffu, j < c1 && key > thr));
      n_eq += __popc(__ballot_sync(0xffffffffu, j < c1 && key == thr));
    }
  }
  __syncthreads();  // wsum is free again
  if (lane == 0) {
    sm->wsum[warp] = n_gt;
    sm->weq[warp] = n_eq;
  }
  __syncthreads();
  // every warp ranks the warps: equal keys before warp w, then kept tokens before warp w
  const int e = sm->weq[lane];
  int e_inc = e;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, e_inc, o);
    if (lane >= o) e_inc += t;
  }
  const int kept_w = sm->wsum[lane] + min(e, max(0, need_eq - (e_inc - e)));
  int k_inc = kept_w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, k_inc, o);
    if (lane >= o) k_inc += t;
  }
  const int tot = __shfl_sync(0xffffffffu, k_inc, 31);
  int eq_seen = __shfl_sync(0xffffffffu, e_inc - e, warp);
  int pos = __shfl_sync(0xffffffffu, k_inc - kept_w, warp);
  if (k > 0) {
    for (int j0 = c0; j0 < c1; j0 += 32) {
      const int j = j0 + lane;
      const uint32_t key = j < c1 ? key_at(j) : 0u;
      const bool is_eq = j < c1 && key == thr;
      const uint32_t b_eq = __ballot_sync(0xffffffffu, is_eq);
      const bool keep = (j < c1 && key > thr) || (is_eq && eq_seen + __popc(b_eq & lt) < need_eq);
      const uint32_t b_keep = __ballot_sync(0xffffffffu, keep);
      if (keep) out[pos + __popc(b_keep & lt)] = j;
      pos += __popc(b_keep);
      eq_seen += __popc(b_eq);
    }
  }
  if (tot != k && threadIdx.x == 0) atomicExch(status, AUDIOKV_EDEVICE);
  for (int i = threadIdx.x; i < W; i += kSelThreads) out[k + i] = P + i;
  __syncthreads();
}

}  // namespace akv
