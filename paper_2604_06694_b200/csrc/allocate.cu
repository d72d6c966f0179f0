// Head-wise budgets in exact integer arithmetic, and their prefix sums: one thread block per request.
//
// Every head gets window + base rows; the remaining rows R of the request's total are
// shared in proportion to S_q = round-half-up(S * 2^24): floors first, heads whose share
// would exceed the rows they have are fixed at that cap and taken out of the pool (and
// the shares recomputed), and the rows the floors leave over go one each to the largest
// remainders, lower head index first. All-zero scores split R evenly.
#include "common.cuh"

namespace akv {
namespace {

constexpr int kAllocThreads = 256;

constexpr int kAllocChunk = 64;  // requests per launch: their totals travel as kernel arguments

struct BudgetArgs {
  int32_t r0;                    // first request of this launch
  int64_t total[kAllocChunk];    // B_r of requests r0, r0 + 1, ...
  int64_t cu_base[kAllocChunk];  // rows kept by the requests before r: sum of their B (budgets add up exactly)
};

__device__ __forceinline__ long long block_sum_ll(long long v, long long* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  long long t = 0;
  for (int w = 0; w < kAllocThreads / 32; ++w) t += red[w];
  return t;
}

__global__ void __launch_bounds__(kAllocThreads)
allocate_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const float* __restrict__ head_scores, BudgetArgs args,
                int32_t* __restrict__ budgets, int32_t* __restrict__ cu_kept, int* __restrict__ status) {
  extern __shared__ long long sm[];
  chain_release();  // the first scoring sweep, which needs nothing from here, may start beside this kernel
  const int N = sh.heads_per_req;
  long long* Sq = sm;            // [N] quantised scores
  long long* tk = Sq + N;        // [N] share above the floor
  long long* rem = tk + N;       // [N] remainders
  int* active = reinterpret_cast<int*>(rem + N);  // [N] 1 while the head is in the pool
  int* give = active + N;                         // [N] 1 when the head receives a left-over row this turn
  __shared__ long long red[kAllocThreads / 32];

  const int r = args.r0 + blockIdx.x;
  const ReqDesc rq = reqs[r];
  const float* S = head_scores + static_cast<int64_t>(r) * N;
  const long long f = static_cast<long long>(sh.window) + sh.base_per_head;
  const long long cap = rq.L - f;
  long long R = args.total[blockIdx.x] - static_cast<long long>(N) * f;

  for (int h = threadIdx.x; h < N; h += kAllocThreads) {
    const double v = static_cast<double>(S[h]);
    long long q = 0;
    if (!(v >= 0.0) || v > 128.0) {
      atomicExch(status, AUDIOKV_EINVAL);  // invalid score: treated as zero
    } else {
      q = static_cast<long long>(floor(v * 16777216.0 + 0.5));
    }
    Sq[h] = q;
    tk[h] = 0;
    active[h] = 1;
  }
  __syncthreads();

  for (int round = 0; round <= N; ++round) {
    long long lsum = 0, lcnt = 0;
    for (int h = threadIdx.x; h < N; h += kAllocThreads)
      if (active[h]) {
        lsum += Sq[h];
        ++lcnt;
      }
    const long long sum = block_sum_ll(lsum, red);
    const long long nA = block_sum_ll(lcnt, red);
    if (nA == 0) break;
    if (sum == 0) {
      // even split by rank inside the pool
      for (int h = threadIdx.x; h < N; h += kAllocThreads)
        if (active[h]) {
          int rank = 0;
          for (int g = 0; g < h; ++g) rank += active[g];
          tk[h] = R / nA + (rank < R % nA ? 1 : 0);
        }
      break;
    }
    long long lover = 0;
    for (int h = threadIdx.x; h < N; h += kAllocThreads)
      if (active[h]) {
        const long long prod = R * Sq[h];  // R < 2^31 and S_q <= 2^31: no overflow
        const long long sh_ = prod / sum;
        tk[h] = sh_;
        rem[h] = prod - sh_ * sum;
        if (sh_ > cap) ++lover;
      }
    const long long n_over = block_sum_ll(lover, red);
    if (n_over > 0) {
      for (int h = threadIdx.x; h < N; h += kAllocThreads)
        if (active[h] && tk[h] > cap) {
          tk[h] = cap;
          active[h] = 0;
        }
      R -= n_over * cap;
      __syncthreads();
      continue;
    }
    long long lgiven = 0;
    for (int h = threadIdx.x; h < N; h += kAllocThreads)
      if (active[h]) lgiven += tk[h];
    long long left = R - block_sum_ll(lgiven, red);
    // hand out the left-over rows by descending remainder, ties by ascending index, skipping full heads
    while (left > 0) {
      long long lelig = 0;
      for (int h = threadIdx.x; h < N; h += kAllocThreads)
        if (active[h] && tk[h] < cap) ++lelig;
      const long long n_elig = block_sum_ll(lelig, red);
      if (n_elig == 0) break;
      for (int h = threadIdx.x; h < N; h += kAllocThreads)
        if (active[h] && tk[h] < cap) {
          long long rank = 0;
          for (int g = 0; g < N; ++g)
            if (active[g] && tk[g] < cap && (rem[g] > rem[h] || (rem[g] == rem[h] && g < h))) ++rank;
          give[h] = rank < left ? 1 : 0;
        } else {
          give[h] = 0;
        }
      __syncthreads();  // the increments are applied after every thread has ranked against the old shares
      for (int h = threadIdx.x; h < N; h += kAllocThreads)
        if (give[h]) tk[h] += 1;
      left -= n_elig < left ? n_elig : left;
      __syncthreads();
    }
    break;
  }
  __syncthreads();
  for (int h = threadIdx.x; h < N; h += kAllocThreads)
    budgets[rq.head_base + h] = static_cast<int32_t>(f + tk[h]);

  // cu_kept: exclusive prefix sum of the budgets in flat head order. The request's first row is known
  // without looking at other requests, because every request keeps exactly total[r] rows.
  const int per = (N + kAllocThreads - 1) / kAllocThreads;
  const int a = min(N, static_cast<int>(threadIdx.x) * per), b = min(N, a + per);
  long long local = 0;
  for (int h = a; h < b; ++h) local += f + tk[h];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long inc = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) red[warp] = inc;
  __syncthreads();
  long long run = args.cu_base[blockIdx.x] + inc - local;
  for (int w = 0; w < warp; ++w) run += red[w];
  for (int h = a; h < b; ++h) {
    cu_kept[rq.head_base + h] = static_cast<int32_t>(run);
    run += f + tk[h];
  }
  if (r == sh.n_req - 1 && threadIdx.x == 0)
    cu_kept[sh.total_heads] = static_cast<int32_t>(args.cu_base[blockIdx.x] + args.total[blockIdx.x]);
}

// Budgets handed in by the caller: a checked copy (each clamped into [W, L] of its request, a clamp being reported
// through the status word) and its exclusive prefix sums. One block; the heads are walked in chunks of the block size.
__global__ void __launch_bounds__(1024)
budget_prefix_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const int32_t* __restrict__ given,
                     int32_t* __restrict__ budgets, int32_t* __restrict__ cu_kept, int* __restrict__ status) {
  __shared__ long long warp_sum[32];
  __shared__ long long carry;
  chain_release();  // the first scoring sweep, which needs nothing from here, may start beside this kernel
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int u0 = 0; u0 < sh.total_heads; u0 += 1024) {
    const int u = u0 + threadIdx.x;
    long long b = 0;
    if (u < sh.total_heads) {
      const int L = reqs[u / sh.heads_per_req].L;
      int g = given[u];
      if (g < sh.window || g > L) {
        atomicExch(status, AUDIOKV_EINVAL);
        g = g < sh.window ? sh.window : L;
      }
      budgets[u] = g;
      b = g;
    }
    long long inc = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    long long before = carry;
    for (int w = 0; w < warp; ++w) before += warp_sum[w];
    if (u < sh.total_heads) cu_kept[u] = static_cast<int32_t>(before + inc - b);
    __syncthreads();
    if (threadIdx.x == 1023) carry = before + inc;
    __syncthreads();
  }
  if (threadIdx.x == 0) cu_kept[sh.total_heads] = static_cast<int32_t>(carry);
}

}  // namespace

cudaError_t launch_budget_prefix(const Shape& sh, const ReqDesc* d_reqs, const int32_t* given, int32_t* budgets,
                                 int32_t* cu_kept, int* status, Launch ln) {
  budget_prefix_kernel<<<1, 1024, 0, ln.stream>>>(sh, d_reqs, given, budgets, cu_kept, status);
  ln.done("budget_prefix");
  return cudaGetLastError();
}

cudaError_t launch_allocate(const Shape& sh, const ReqDesc* d_reqs, const float* head_scores,
                            const int64_t* h_total_budget, int32_t* budgets, int32_t* cu_kept, int* status,
                            Launch ln) {
  int64_t all = 0;
  for (int r = 0; r < sh.n_req; ++r) all += h_total_budget[r];
  if (all > 0x7fffffffLL) return cudaErrorInvalidValue;  // cu_kept is int32
  const size_t smem = static_cast<size_t>(sh.heads_per_req) * (3 * sizeof(long long) + 2 * sizeof(int));
  cudaError_t e = cudaFuncSetAttribute(allocate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int64_t rows = 0;
  for (int r0 = 0; r0 < sh.n_req; r0 += kAllocChunk) {
    const int n = sh.n_req - r0 < kAllocChunk ? sh.n_req - r0 : kAllocChunk;
    BudgetArgs args{};
    args.r0 = r0;
    for (int i = 0; i < n; ++i) {
      args.total[i] = h_total_budget[r0 + i];
      args.cu_base[i] = rows;
      rows += h_total_budget[r0 + i];
    }
    allocate_kernel<<<n, kAllocThreads, smem, ln.stream>>>(sh, d_reqs, head_scores, args, budgets, cu_kept, status);
    ln.done("allocate");
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace akv
