// Per-head top-k by radix select, ordered compaction of the kept indices, and the
// vectorised gather of the kept K and V rows into the compacted cache.
#include "common.cuh"
#include "select.cuh"

namespace akv {
namespace {

// One block per head: the head's keys staged once in shared memory when they fit, then select_topk.
__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const float* __restrict__ smoothed,
              const int32_t* __restrict__ budgets, const int32_t* __restrict__ cu_kept,
              int32_t* __restrict__ kept_idx, int smem_keys, int* __restrict__ status) {
  extern __shared__ uint32_t skeys[];
  __shared__ SelectSmem ssm;

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
    const bool staged = P <= smem_keys;
    __syncthreads();
    if (staged)
      for (int j = threadIdx.x; j < P; j += kSelThreads) skeys[j] = score_key(s[j]);
    __syncthreads();
    if (staged)
      select_topk([&](int j) -> uint32_t { return skeys[j]; }, P, W, k, kept_idx + cu_kept[u], &ssm, status);
    else
      select_topk([&](int j) -> uint32_t { return score_key(s[j]); }, P, W, k, kept_idx + cu_kept[u], &ssm, status);
  }
}

// Copies the kept rows. A warp takes eight output rows at a time: lanes 0-7 look up the head of one row each
// (bisection in cu_kept) and its source row; then all lanes copy 16-byte chunks, K chunks first, V chunks after,
// eight independent loads in flight per lane before the stores. log2_chunks: log2 of the chunks per row.
// Rows are read and written once: both sides carry the streaming hint, so that the hundreds of megabytes that pass
// through leave the small, reused state of the pass (tables, scores, statistics, the kernels' code) in L2. Measured
// on the 28-layer L = 8192 pass: the smoothing kernel of the next pass took 35 us instead of 43.
constexpr int kGatherRows = 8;

__global__ void __launch_bounds__(256, 3)  // three blocks per SM: at most 80 registers per thread
gather_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const int32_t* __restrict__ cu_kept,
              const int32_t* __restrict__ kept_idx, const uint4* __restrict__ k, const uint4* __restrict__ v,
              uint4* __restrict__ k_out, uint4* __restrict__ v_out, int log2_chunks, int elems_per_chunk,
              int head_begin, int head_end) {
  // Launched the ordinary way, after the smoothing kernel has finished: brought in early (programmatic dependent
  // launch) its blocks only sat on the SMs that finished their heads first, and a ragged batch ran 7 % slower.
  chain_release();  // the next pass's first scoring sweep may be set up while this kernel drains
  const int64_t first_row = cu_kept[head_begin];  // the rows of heads [head_begin, head_end)
  const int64_t total_rows = cu_kept[head_end];
  const int64_t n_batches = (total_rows - first_row + kGatherRows - 1) / kGatherRows;
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
  const int64_t n_warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  const int chunks = 1 << log2_chunks;
  for (int64_t bt = warp0; bt < n_batches; bt += n_warps) {
    const int64_t row0 = first_row + bt * kGatherRows;
    int64_t my_src = 0;  // lane i < 8: first 16-byte chunk of the source row of output row row0 + i
    if (lane < kGatherRows && row0 + lane < total_rows) {
      const int64_t row = row0 + lane;
      int lo = head_begin, hi = head_end;  // largest u with cu_kept[u] <= row
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(cu_kept + mid) <= row) lo = mid; else hi = mid;
      }
      const int u = lo;
      const ReqDesc rq = reqs[u / sh.heads_per_req];
      const int lh = u - rq.head_base;
      const int l = lh / sh.n_kv_heads, h = lh - l * sh.n_kv_heads;
      const int tok = __ldg(kept_idx + row);
      my_src = (l * sh.kv_stride_layer + h * sh.kv_stride_head + kv_token_offset(sh, rq, u / sh.heads_per_req, tok)) /
               elems_per_chunk;
    }
    const int n_rows = static_cast<int>(min(static_cast<int64_t>(kGatherRows), total_rows - row0));
    int64_t so[kGatherRows];  // every lane gets the eight source rows (all lanes take part in the shuffles)
#pragma unroll
    for (int i = 0; i < kGatherRows; ++i) so[i] = __shfl_sync(0xffffffffu, my_src, i);
    for (int c0 = lane; c0 < 2 * chunks; c0 += 32) {
      const bool is_v = c0 >= chunks;
      const int c = c0 & (chunks - 1);
      const uint4* src = is_v ? v : k;
      uint4* dst = (is_v ? v_out : k_out) + (row0 << log2_chunks) + c;
      uint4 val[kGatherRows];
#pragma unroll
      for (int i = 0; i < kGatherRows; ++i)
        if (i < n_rows) val[i] = __ldcs(src + so[i] + c);
#pragma unroll
      for (int i = 0; i < kGatherRows; ++i)
        if (i < n_rows) __stcs(dst + (static_cast<int64_t>(i) << log2_chunks), val[i]);
    }
  }
}

}  // namespace

cudaError_t launch_select(const Shape& sh, const ReqDesc* d_reqs, const float* smoothed, const int32_t* budgets,
                          const int32_t* cu_kept, int32_t* kept_idx, int max_P, int* status, Launch ln) {
  const int smem_keys = max_P <= 48 * 1024 ? max_P : 48 * 1024;
  const size_t smem = static_cast<size_t>(smem_keys) * sizeof(uint32_t);
  cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int max_grid = device_sm_count() * 4;
  const int grid = sh.total_heads < max_grid ? sh.total_heads : max_grid;
  select_kernel<<<grid, kSelThreads, smem, ln.stream>>>(sh, d_reqs, smoothed, budgets, cu_kept, kept_idx, smem_keys,
                                                        status);
  ln.done("select");
  return cudaGetLastError();
}

cudaError_t launch_gather(const Shape& sh, const ReqDesc* d_reqs, const int32_t* cu_kept, const int32_t* kept_idx,
                          const void* k, const void* v, void* k_out, void* v_out, int head_begin, int head_end,
                          Launch ln) {
  const int esize = sh.dtype == AUDIOKV_F32 ? 4 : 2;
  const int elems_per_chunk = 16 / esize;
  const int chunks_per_row = sh.head_dim / elems_per_chunk;  // 8 .. 64: head_dim is 64, 128 or 256
  int log2_chunks = 0;
  while ((1 << log2_chunks) < chunks_per_row) ++log2_chunks;
  gather_kernel<<<dim3(device_sm_count() * 8), dim3(256), 0, ln.stream>>>(sh, d_reqs, cu_kept, kept_idx, (const uint4*)k, (const uint4*)v,
                                                         (uint4*)k_out, (uint4*)v_out, log2_chunks, elems_per_chunk,
                                                         head_begin, head_end);
  cudaError_t e = cudaGetLastError();
  ln.done("gather");
  return e;
}

}  // namespace akv
