// Offline head score: for every decode step and head, the top-K tokens of the attention row, how many of them
// fall inside the audio span of the word generated at that step, and the mean of that ratio over the steps.
// One block per (step, head) pair (grid-stride): the radix select of select.cuh on the row read straight from
// global memory, the K indices into shared memory, a count against the span, one integer atomic per pair.
#include "common.cuh"
#include "select.cuh"

namespace akv {
namespace {

constexpr int kHitMaxK = 1024;

__global__ void __launch_bounds__(kSelThreads, 1)
hit_count_kernel(const float* __restrict__ attn, int n_steps, int n_heads, int64_t row_stride,
                 const int32_t* __restrict__ row_len, const int32_t* __restrict__ span, int top_k,
                 int32_t* __restrict__ counts, int* __restrict__ status) {
  __shared__ SelectSmem ssm;
  __shared__ int32_t top_idx[kHitMaxK];
  __shared__ int s_hits;
  const int n_pairs = n_steps * n_heads;
  for (int pair = blockIdx.x; pair < n_pairs; pair += gridDim.x) {
    const int t = pair / n_heads, a = pair - t * n_heads;
    const int L = row_len[t];
    const float* row = attn + static_cast<int64_t>(pair) * row_stride;
    const int k = min(top_k, L);
    __syncthreads();
    if (threadIdx.x == 0) s_hits = 0;
    // no window here (W = 0): select_topk leaves the k indices in ascending token order
    select_topk([&](int j) -> uint32_t { return score_key(row[j]); }, L, 0, k, top_idx, &ssm, status);
    const int lo = span[2 * t], hi = span[2 * t + 1];
    int c = 0;
    for (int i = threadIdx.x; i < k; i += kSelThreads) c += top_idx[i] >= lo && top_idx[i] <= hi;
    c = __reduce_add_sync(0xffffffffu, c);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&s_hits, c);
    __syncthreads();
    if (threadIdx.x == 0 && s_hits) atomicAdd(counts + a, s_hits);
  }
}

__global__ void hit_ratio_kernel(const int32_t* __restrict__ counts, int n_heads, int n_steps, int top_k,
                                 float* __restrict__ s_hit) {
  const int a = blockIdx.x * blockDim.x + threadIdx.x;
  if (a < n_heads)
    s_hit[a] = static_cast<float>(static_cast<double>(counts[a]) / (static_cast<double>(top_k) * n_steps));
}

}  // namespace

cudaError_t launch_hit_score(const float* attn, int n_steps, int n_heads, int64_t row_stride, const int32_t* row_len,
                             const int32_t* span, int top_k, int32_t* counts, float* s_hit, int* status, Launch ln) {
  cudaError_t e = cudaMemsetAsync(counts, 0, sizeof(int32_t) * n_heads, ln.stream);
  if (e != cudaSuccess) return e;
  const int64_t n_pairs = static_cast<int64_t>(n_steps) * n_heads;
  const int max_grid = device_sm_count() * 2;
  const int grid = static_cast<int>(n_pairs < max_grid ? n_pairs : max_grid);
  hit_count_kernel<<<grid, kSelThreads, 0, ln.stream>>>(attn, n_steps, n_heads, row_stride, row_len, span, top_k, counts,
                                                        status);
  ln.done("hit_count");
  hit_ratio_kernel<<<(n_heads + 255) / 256, 256, 0, ln.stream>>>(counts, n_heads, n_steps, top_k, s_hit);
  ln.done("hit_ratio");
  return cudaGetLastError();
}

}  // namespace akv
