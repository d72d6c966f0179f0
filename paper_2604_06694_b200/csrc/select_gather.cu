// Per-head top-k by radix select, ordered compaction of the kept indices, and the
// vectorised gather of the kept K and V rows into the compacted cache.
#include "common.cuh"

namespace akv {
namespace {

constexpr int kSelThreads = 1024;

// Order-preserving map float -> uint32 (larger float, larger key); -0 and +0 share a key.
__device__ __forceinline__ uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

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

// One block per head: k-th largest key by four 8-bit radix passes over the head's scores
// (staged once in shared memory when they fit), then the kept indices in ascending order.
__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const float* __restrict__ smoothed,
              const int32_t* __restrict__ budgets, const int32_t* __restrict__ cu_kept,
              int32_t* __restrict__ kept_idx, int smem_keys, int* __restrict__ status) {
  extern __shared__ uint32_t skeys[];
  __shared__ int hist[256];
  __shared__ int wsum[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_want;

  for (int u = blockIdx.x; u < sh.total_heads; u += gridDim.x) {
    const int r = u / sh.heads_per_req;
    const ReqDesc rq = reqs[r];
    const int P = rq.P, W = sh.window;
    const float* s = smoothed + rq.score_offset + static_cast<int64_t>(u - rq.head_base) * P;
    int k = budgets[u] - W;
    if (k < 0 || k > P) {
      if (threadIdx.x == 0) atomicExch(status, AUDIOKV_EDEVICE);
      k = k < 0 ? 0 : P;
    }
    int32_t* out = kept_idx + cu_kept[u];
    const bool staged = P <= smem_keys;
    __syncthreads();
    if (staged)
      for (int j = threadIdx.x; j < P; j += kSelThreads) skeys[j] = score_key(s[j]);
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return staged ? skeys[j] : score_key(s[j]); };

    uint32_t thr = 0;     // key of the k-th largest element
    int need_eq = 0;      // how many elements equal to thr are kept (those with the lowest indices)
    if (k > 0 && k < P) {
      if (threadIdx.x == 0) {
        s_prefix = 0u;
        s_want = k;
      }
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int b = threadIdx.x; b < 256; b += kSelThreads) hist[b] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
        for (int j = threadIdx.x; j < P; j += kSelThreads) {
          const uint32_t key = key_at(j);
          if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
          int want = s_want, b = 255;
          for (; b > 0; --b) {
            if (hist[b] >= want) break;
            want -= hist[b];
          }
          s_prefix = prefix | (static_cast<uint32_t>(b) << shift);
          s_want = want;
        }
        __syncthreads();
      }
      thr = s_prefix;
      need_eq = s_want;
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
    const int eq_before = block_excl_scan_int(n_eq, wsum, &tot);
    int my_eq_kept = min(n_eq, max(0, need_eq - eq_before));
    if (k == 0) my_eq_kept = 0;
    int pos = block_excl_scan_int(n_gt + my_eq_kept, wsum, &tot);
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
}

// Copies the kept rows. One 16-byte chunk of a K row and of the matching V row per thread
// and step; the head of an output row is found by bisection in cu_kept.
__global__ void __launch_bounds__(256)
gather_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const int32_t* __restrict__ cu_kept,
              const int32_t* __restrict__ kept_idx, const uint4* __restrict__ k, const uint4* __restrict__ v,
              uint4* __restrict__ k_out, uint4* __restrict__ v_out, int chunks_per_row, int elems_per_chunk) {
  const int64_t total_rows = cu_kept[sh.total_heads];
  const int64_t n_items = total_rows * chunks_per_row;
  for (int64_t it = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; it < n_items;
       it += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t row = it / chunks_per_row;
    const int c = static_cast<int>(it - row * chunks_per_row);
    int lo = 0, hi = sh.total_heads;  // largest u with cu_kept[u] <= row
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cu_kept[mid] <= row) lo = mid; else hi = mid;
    }
    const int u = lo;
    const int r = u / sh.heads_per_req;
    const ReqDesc rq = reqs[r];
    const int lh = u - rq.head_base;
    const int l = lh / sh.n_kv_heads, h = lh - l * sh.n_kv_heads;
    const int tok = kept_idx[row];
    const int64_t src_elem = rq.kv_offset + l * sh.kv_stride_layer + h * sh.kv_stride_head + tok * sh.kv_stride_tok;
    const int64_t src = src_elem / elems_per_chunk + c;
    const uint4 kv = __ldg(k + src);
    const uint4 vv = __ldg(v + src);
    k_out[it] = kv;
    v_out[it] = vv;
  }
}

}  // namespace

cudaError_t launch_select(const Shape& sh, const ReqDesc* d_reqs, const float* smoothed, const int32_t* budgets,
                          const int32_t* cu_kept, int32_t* kept_idx, int max_P, int* status, Launch ln) {
  const int smem_keys = max_P <= 48 * 1024 ? max_P : 48 * 1024;
  const size_t smem = static_cast<size_t>(smem_keys) * sizeof(uint32_t);
  cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = sh.total_heads < 148 * 4 ? sh.total_heads : 148 * 4;
  select_kernel<<<grid, kSelThreads, smem, ln.stream>>>(sh, d_reqs, smoothed, budgets, cu_kept, kept_idx, smem_keys,
                                                        status);
  ln.done("select");
  return cudaGetLastError();
}

cudaError_t launch_gather(const Shape& sh, const ReqDesc* d_reqs, const int32_t* cu_kept, const int32_t* kept_idx,
                          const void* k, const void* v, void* k_out, void* v_out, Launch ln) {
  const int esize = sh.dtype == AUDIOKV_F32 ? 4 : 2;
  const int elems_per_chunk = 16 / esize;
  const int chunks_per_row = sh.head_dim / elems_per_chunk;
  gather_kernel<<<148 * 8, 256, 0, ln.stream>>>(sh, d_reqs, cu_kept, kept_idx, (const uint4*)k, (const uint4*)v,
                                                 (uint4*)k_out, (uint4*)v_out, chunks_per_row, elems_per_chunk);
  ln.done("gather");
  return cudaGetLastError();
}

}  // namespace akv
