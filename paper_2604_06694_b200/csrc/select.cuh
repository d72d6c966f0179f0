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
// the k-th largest key; the bin that holds it is located by a block-wide scan over the counts.
template <typename KeyAt>
__device__ __forceinline__ void select_topk(KeyAt key_at, int P, int W, int k, int32_t* __restrict__ out,
                                            SelectSmem* sm, int* __restrict__ status) {
  uint32_t thr = 0;  // key of the k-th largest element
  int need_eq = 0;   // how many elements equal to thr are kept (those with the lowest indices)
  if (k > 0 && k < P) {
    __syncthreads();
    if (threadIdx.x == 0) {
      sm->prefix = 0u;
      sm->want = k;
    }
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;
      const int bits = pass == 2 ? 10 : 11;
      const uint32_t dmask = (1u << bits) - 1u;
      for (int b = threadIdx.x; b < kSelBins; b += kSelThreads) sm->hist[b] = 0;
      __syncthreads();
      const uint32_t prefix = sm->prefix;
      const int want = sm->want;
      const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + bits));
      for (int j = threadIdx.x; j < P; j += kSelThreads) {
        const uint32_t key = key_at(j);
        if ((key & pmask) == prefix) atomicAdd(&sm->hist[(key >> shift) & dmask], 1);
      }
      __syncthreads();
      // thread t owns bins 2047 - 2t and 2046 - 2t (descending): `above` counts the keys in higher bins
      const int b_hi = kSelBins - 1 - 2 * static_cast<int>(threadIdx.x), b_lo = b_hi - 1;
      const int c_hi = sm->hist[b_hi], c_lo = sm->hist[b_lo];
      int tot;
      const int above = block_excl_scan_int(c_hi + c_lo, sm->wsum, &tot);
      if (above < want && want <= above + c_hi) {
        sm->prefix = prefix | (static_cast<uint32_t>(b_hi) << shift);
        sm->want = want - above;
      } else if (above + c_hi < want && want <= above + c_hi + c_lo) {
        sm->prefix = prefix | (static_cast<uint32_t>(b_lo) << shift);
        sm->want = want - above - c_hi;
      }
      __syncthreads();
    }
    thr = sm->prefix;
    need_eq = sm->want;
  } else if (k == P) {
    thr = 0u;
    need_eq = P;  // every key is >= 0: keep all
  }

  // ordered compaction: thread t owns the contiguous index range [a, b)
  const int per = (P + kSelThreads - 1) / kSelThreads;
  const int a = min(P, static_cast<int>(threadIdx.x) * per), b = min(P, a + per);
  int n_eq = 0, n_gt = 0;
  if (k > 0) {
    for (int j = a; j < b; ++j) {
      const uint32_t key = key_at(j);
      n_eq += key == thr;
      n_gt += key > thr;
    }
  }
  int tot;
  const int eq_before = block_excl_scan_int(n_eq, sm->wsum, &tot);
  int my_eq_kept = min(n_eq, max(0, need_eq - eq_before));
  if (k == 0) my_eq_kept = 0;
  int pos = block_excl_scan_int(n_gt + my_eq_kept, sm->wsum, &tot);
  if (k > 0) {
    int eq_seen = eq_before;
    for (int j = a; j < b; ++j) {
      const uint32_t key = key_at(j);
      bool keep = key > thr;
      if (key == thr) {
        keep = eq_seen < need_eq;
        ++eq_seen;
      }
      if (keep) out[pos++] = j;
    }
  }
  if (tot != k && threadIdx.x == 0) atomicExch(status, AUDIOKV_EDEVICE);
  for (int i = threadIdx.x; i < W; i += kSelThreads) out[k + i] = P + i;
  __syncthreads();
}

}  // namespace akv
