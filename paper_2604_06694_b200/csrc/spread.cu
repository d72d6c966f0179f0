// Selection spread: where along the prefix the kept tokens of a request's heads fall. Token j of a prefix of P
// tokens belongs to stretch floor(j * n_bins / P); hist[r][b] counts the kept prefix tokens of all heads of request r
// in stretch b (window tokens are not counted). Two summaries per request: balance = normalised entropy of the
// histogram, peak = busiest stretch against the mean stretch.
// One block per head builds the head's histogram in shared memory and adds it to the request's; one block per
// request then reduces the histogram in double precision.
#include "common.cuh"

namespace akv {
namespace {

constexpr int kSpreadThreads = 256;
constexpr int kSpreadMaxBins = 4096;

__global__ void __launch_bounds__(kSpreadThreads)
spread_hist_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const int32_t* __restrict__ kept_idx,
                   const int32_t* __restrict__ cu_kept, int n_bins, int32_t* __restrict__ hist,
                   int* __restrict__ status) {
  __shared__ int32_t h[kSpreadMaxBins];
  const int u = blockIdx.x;
  const int r = u / sh.heads_per_req;
  const int P = reqs[r].P;
  for (int b = threadIdx.x; b < n_bins; b += kSpreadThreads) h[b] = 0;
  __syncthreads();
  const int a = cu_kept[u], e = cu_kept[u + 1];
  for (int i = a + threadIdx.x; i < e; i += kSpreadThreads) {
    const int j = kept_idx[i];
    if (j < 0 || j >= reqs[r].L) {
      atomicExch(status, AUDIOKV_EDEVICE);  // not an index of this head: skipped
      continue;
    }
    if (j < P) atomicAdd(&h[static_cast<long long>(j) * n_bins / P], 1);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < n_bins; b += kSpreadThreads)
    if (h[b]) atomicAdd(hist + static_cast<int64_t>(r) * n_bins + b, h[b]);
}

__global__ void __launch_bounds__(kSpreadThreads)
spread_stats_kernel(const int32_t* __restrict__ hist, int n_bins, float* __restrict__ stats) {
  __shared__ long long s_tot[kSpreadThreads / 32];
  __shared__ int s_top[kSpreadThreads / 32];
  __shared__ double s_ent[kSpreadThreads / 32];
  const int32_t* hr = hist + static_cast<int64_t>(blockIdx.x) * n_bins;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long tot = 0;
  int top = 0;
  for (int b = threadIdx.x; b < n_bins; b += kSpreadThreads) {
    tot += hr[b];
    top = max(top, hr[b]);
  }
  for (int o = 16; o > 0; o >>= 1) {
    tot += __shfl_xor_sync(0xffffffffu, tot, o);
    top = max(top, __shfl_xor_sync(0xffffffffu, top, o));
  }
  if (lane == 0) {
    s_tot[warp] = tot;
    s_top[warp] = top;
  }
  __syncthreads();
  tot = 0;
  top = 0;
  for (int w = 0; w < kSpreadThreads / 32; ++w) {
    tot += s_tot[w];
    top = max(top, s_top[w]);
  }
  double ent = 0.0;
  if (tot > 0)
    for (int b = threadIdx.x; b < n_bins; b += kSpreadThreads)
      if (hr[b] > 0) {
        const double p = static_cast<double>(hr[b]) / static_cast<double>(tot);
        ent -= p * log(p);
      }
  for (int o = 16; o > 0; o >>= 1) ent += __shfl_xor_sync(0xffffffffu, ent, o);
  if (lane == 0) s_ent[warp] = ent;
  __syncthreads();
  if (threadIdx.x == 0) {
    ent = 0.0;
    for (int w = 0; w < kSpreadThreads / 32; ++w) ent += s_ent[w];
    float balance = 0.f, peak = 0.f;
    if (tot > 0) {
      peak = static_cast<float>(static_cast<double>(top) * n_bins / static_cast<double>(tot));
      if (n_bins > 1) balance = static_cast<float>(ent / log(static_cast<double>(n_bins)));
    }
    stats[2 * blockIdx.x] = balance;
    stats[2 * blockIdx.x + 1] = peak;
  }
}

}  // namespace

cudaError_t launch_selection_spread(const Shape& sh, const ReqDesc* d_reqs, const int32_t* kept_idx,
                                    const int32_t* cu_kept, int n_bins, int32_t* hist, float* stats, int* status,
                                    Launch ln) {
  if (n_bins < 1 || n_bins > kSpreadMaxBins) return cudaErrorInvalidValue;
  cudaError_t e = cudaMemsetAsync(hist, 0, sizeof(int32_t) * static_cast<size_t>(sh.n_req) * n_bins, ln.stream);
  if (e != cudaSuccess) return e;
  spread_hist_kernel<<<sh.total_heads, kSpreadThreads, 0, ln.stream>>>(sh, d_reqs, kept_idx, cu_kept, n_bins, hist,
                                                                       status);
  ln.done("spread_hist");
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  spread_stats_kernel<<<sh.n_req, kSpreadThreads, 0, ln.stream>>>(hist, n_bins, stats);
  ln.done("spread_stats");
  return cudaGetLastError();
}

}  // namespace akv
