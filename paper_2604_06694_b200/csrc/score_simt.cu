// Importance scores on the fp32 FMA pipe, for any element type.
//
// This is the path for fp32 inputs (which must not be rounded to TF32) and the
// fallback for shapes the tensor-core kernels do not take. Two sweeps over the keys:
//   sweep 1  per (head, key slab): running max and sum of exp2 of every window row,
//   sweep 2  per (head, key slab): merge the slabs' statistics, then for every prefix
//            key sum exp2(z - max - log2 sum) over the rows.
// Logits are kept in base 2 (scale * log2 e folded into one multiply).
#include "common.cuh"

namespace akv {
namespace {

constexpr int kTile = 64;      // keys per tile and rows per row chunk
constexpr int kThreads = 256;  // 16 x 16 threads, 4 x 4 logits each

template <typename T>
__device__ __forceinline__ float4 load4(const T* p);
template <>
__device__ __forceinline__ float4 load4<float>(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
template <>
__device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
  uint2 raw = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&raw.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&raw.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}

struct HeadCoord {
  int r, l, h;
};
__device__ __forceinline__ HeadCoord head_coord(const Shape& sh, int u) {
  HeadCoord c;
  c.r = u / sh.heads_per_req;
  int lh = u - c.r * sh.heads_per_req;
  c.l = lh / sh.n_kv_heads;
  c.h = lh - c.l * sh.n_kv_heads;
  return c;
}

// Stages `kTile` rows of D elements as fp32 into smem (row stride D + 4); rows >= n_valid are zero.
template <typename T, int D, typename RowPtr>
__device__ __forceinline__ void stage_rows(float* smem, int n_valid, RowPtr row_ptr) {
  constexpr int C4 = D / 4;
  for (int idx = threadIdx.x; idx < kTile * C4; idx += kThreads) {
    int row = idx / C4, c4 = idx - row * C4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row < n_valid) v = load4<T>(row_ptr(row) + c4 * 4);
    *reinterpret_cast<float4*>(smem + row * (D + 4) + c4 * 4) = v;
  }
}

// acc[a][b] = <Q row ty + 16 a, K row tx + 16 b>
template <int D>
__device__ __forceinline__ void tile_dot(const float* Qs, const float* Ks, int ty, int tx, float acc[4][4]) {
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
  for (int t = 0; t < D; t += 4) {
    float4 qv[4], kv[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) qv[a] = *reinterpret_cast<const float4*>(Qs + (ty + 16 * a) * (D + 4) + t);
#pragma unroll
    for (int b = 0; b < 4; ++b) kv[b] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * b) * (D + 4) + t);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        acc[a][b] = fmaf(qv[a].x, kv[b].x, acc[a][b]);
        acc[a][b] = fmaf(qv[a].y, kv[b].y, acc[a][b]);
        acc[a][b] = fmaf(qv[a].z, kv[b].z, acc[a][b]);
        acc[a][b] = fmaf(qv[a].w, kv[b].w, acc[a][b]);
      }
  }
}

// SWEEP = 1: row statistics; SWEEP = 2: column sums.
template <typename T, int D, int SWEEP>
__global__ void __launch_bounds__(kThreads) score_simt_kernel(Shape sh, const ReqDesc* __restrict__ reqs,
                                                              const T* __restrict__ q, const T* __restrict__ k,
                                                              float* __restrict__ scores, float2* __restrict__ stats,
                                                              int n_slab, int slab_keys) {
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = Qs + kTile * (D + 4);
  float* Zt = Ks + kTile * (D + 4);      // [kTile][kTile + 1]
  float* rowA = Zt + kTile * (kTile + 1);  // sweep 1: running max; sweep 2: max + log2 sum
  float* rowB = rowA + sh.window * sh.group;  // sweep 1: running sum; sweep 2: partial column sums [4][kTile]

  const int u = blockIdx.x / n_slab, slab = blockIdx.x - u * n_slab;  // one block per (head, slab), heads outermost
  const HeadCoord hc = head_coord(sh, u);
  const ReqDesc rq = reqs[hc.r];
  const int R = sh.window * sh.group, G = sh.group;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const int j0 = slab * slab_keys;
  const int j_end = SWEEP == 1 ? rq.L : rq.P;  // sweep 2 only needs the prefix keys
  const int j1 = min(j_end, j0 + slab_keys);
  float2* my_stats = stats + (static_cast<int64_t>(u) * n_slab + slab) * R;

  const T* kbase = k + hc.l * sh.kv_stride_layer + hc.h * sh.kv_stride_head;  // the token term: kv_token_offset
  const T* qbase = q + rq.q_offset + hc.l * sh.q_stride_layer + static_cast<int64_t>(hc.h) * G * sh.q_stride_head;

  if (SWEEP == 1) {
    for (int r = threadIdx.x; r < R; r += kThreads) {
      rowA[r] = -INFINITY;
      rowB[r] = 0.f;
    }
  } else {
    const float2* hs = stats + static_cast<int64_t>(u) * n_slab * R;
    for (int r = threadIdx.x; r < R; r += kThreads) {
      float M = -INFINITY;
      for (int s = 0; s < n_slab; ++s) M = fmaxf(M, hs[static_cast<int64_t>(s) * R + r].x);
      float Z = 0.f;
      for (int s = 0; s < n_slab; ++s) {
        float2 st = hs[static_cast<int64_t>(s) * R + r];
        if (st.y > 0.f) Z += st.y * exp2f(st.x - M);
      }
      rowA[r] = M + log2f(Z);
    }
  }
  __syncthreads();

  for (int kt = j0; kt < j1; kt += kTile) {
    const int nk = min(kTile, j1 - kt);
    stage_rows<T, D>(Ks, nk, [&](int row) { return kbase + kv_token_offset(sh, rq, hc.r, kt + row); });
    float colsum = 0.f;  // sweep 2, threads 0..63
    for (int rc = 0; rc < R; rc += kTile) {
      const int nr = min(kTile, R - rc);
      __syncthreads();  // Qs, Zt free
      stage_rows<T, D>(Qs, nr, [&](int row) {
        int rr = rc + row;
        int i = rr / G, g = rr - i * G;
        return qbase + i * sh.q_stride_tok + g * sh.q_stride_head;
      });
      __syncthreads();
      float acc[4][4];
      tile_dot<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int row = ty + 16 * a, rr = rc + row;
        const int i = rr / G;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int key = tx + 16 * b, j = kt + key;
          float z = acc[a][b] * sh.scale_log2e;
          if (SWEEP == 1) {
            bool ok = rr < R && key < nk && j <= rq.P + i;
            Zt[row * (kTile + 1) + key] = ok ? z : -INFINITY;
          } else {
            bool ok = rr < R && key < nk;
            Zt[row * (kTile + 1) + key] = ok ? exp2f(z - rowA[rr < R ? rr : 0]) : 0.f;
          }
        }
      }
      __syncthreads();
      if (SWEEP == 1) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int row = warp; row < nr; row += kThreads / 32) {
          float z0 = Zt[row * (kTile + 1) + lane], z1 = Zt[row * (kTile + 1) + lane + 32];
          float m = fmaxf(z0, z1);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          if (m > -INFINITY) {
            const float m_old = rowA[rc + row];
            const float m_new = fmaxf(m_old, m);
            float e = exp2f(z0 - m_new) + exp2f(z1 - m_new);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
            if (lane == 0) {
              rowB[rc + row] = rowB[rc + row] * exp2f(m_old - m_new) + e;
              rowA[rc + row] = m_new;
            }
          }
        }
      } else {
        const int key = threadIdx.x & 63, part = threadIdx.x >> 6;
        float sacc = 0.f;
#pragma unroll
        for (int rr = 0; rr < 16; ++rr) sacc += Zt[(part * 16 + rr) * (kTile + 1) + key];
        rowB[part * kTile + key] = sacc;
        __syncthreads();
        if (threadIdx.x < kTile)
          colsum += (rowB[threadIdx.x] + rowB[kTile + threadIdx.x]) + (rowB[2 * kTile + threadIdx.x] + rowB[3 * kTile + threadIdx.x]);
      }
    }
    if (SWEEP == 2 && threadIdx.x < nk) {
      scores[rq.score_offset + (static_cast<int64_t>(hc.l) * sh.n_kv_heads + hc.h) * rq.P + kt + threadIdx.x] = colsum;
    }
    __syncthreads();  // Ks free
  }
  if (SWEEP == 1) {
    __syncthreads();
    for (int r = threadIdx.x; r < R; r += kThreads) my_stats[r] = make_float2(rowA[r], rowB[r]);
  }
}

template <typename T, int D>
cudaError_t launch_typed(const Shape& sh, const ReqDesc* d_reqs, const void* q, const void* k, float* scores,
                         float2* stats_ws, int n_slab, int slab_keys, Launch ln) {
  const int R = sh.window * sh.group;
  const int rows_extra = R > 4 * kTile ? R : 4 * kTile;
  size_t smem = sizeof(float) * (2 * kTile * (D + 4) + kTile * (kTile + 1) + R + rows_extra);
  auto k1 = score_simt_kernel<T, D, 1>;
  auto k2 = score_simt_kernel<T, D, 2>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if (static_cast<int64_t>(n_slab) * sh.total_heads > 0x7fffffffLL) return cudaErrorNotSupported;
  dim3 grid(static_cast<unsigned>(n_slab) * static_cast<unsigned>(sh.total_heads));
  k1<<<grid, kThreads, smem, ln.stream>>>(sh, d_reqs, (const T*)q, (const T*)k, scores, stats_ws, n_slab, slab_keys);
  ln.done("score_simt_stats");
  k2<<<grid, kThreads, smem, ln.stream>>>(sh, d_reqs, (const T*)q, (const T*)k, scores, stats_ws, n_slab, slab_keys);
  ln.done("score_simt_colsum");
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_simt(const Shape& sh, const ReqDesc* d_reqs, const void* q, const void* k, float* scores,
                              float2* stats_ws, int n_slab, int slab_keys, Launch ln) {
#define AKV_CASE(T, D) return launch_typed<T, D>(sh, d_reqs, q, k, scores, stats_ws, n_slab, slab_keys, ln)
  if (sh.dtype == AUDIOKV_F32) {
    if (sh.head_dim == 64) AKV_CASE(float, 64);
    if (sh.head_dim == 128) AKV_CASE(float, 128);
    if (sh.head_dim == 256) AKV_CASE(float, 256);
  } else {
    if (sh.head_dim == 64) AKV_CASE(__nv_bfloat16, 64);
    if (sh.head_dim == 128) AKV_CASE(__nv_bfloat16, 128);
    if (sh.head_dim == 256) AKV_CASE(__nv_bfloat16, 256);
  }
#undef AKV_CASE
  return cudaErrorInvalidValue;
}

}  // namespace akv

// ---------------------------------------------------------------------------------------
// Scoring without any allocation.
//
// Some hosts of this library may not allocate device memory at the moment they need the
// scores: code that runs inside a memory-pool or arena whose owner forbids cudaMalloc once
// serving has started, plug-ins that are handed a stream and buffers but no allocator, and
// callers that must not risk the implicit device synchronisation an allocation can cause.
// For them the scratch of the two-sweep scoring (the per-slab row statistics) and the small
// request table live in one fixed array that is part of the library image: every GPU that
// loads the library holds kNoAllocBytes of it until the process exits.
#include <mutex>

namespace akv {
namespace {

constexpr size_t kNoAllocBytes = 8u << 20;     // 8 MiB per GPU, fixed
constexpr size_t kNoAllocTableBytes = 4096;    // request table at the front, statistics after it
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

std::mutex g_noalloc_mu;
void* g_noalloc_ptr[kNoAllocMaxDevices] = {};  // device address of the array, per device ordinal

// The request table reaches the scratch as a kernel argument (2.5 KB, copied at launch): no host
// buffer has to outlive the call.
constexpr int kNoAllocMaxReq = 64;
struct NoAllocTable {
  ReqDesc r[kNoAllocMaxReq];
};
__global__ void noalloc_table_kernel(const NoAllocTable t, int n, ReqDesc* dst) {
  if (threadIdx.x < n) dst[threadIdx.x] = t.r[threadIdx.x];
}

// The array's name is only a host-side handle; kernels need the address the runtime reports
// for the current device.
cudaError_t noalloc_scratch(int device, void** out) {
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (!g_noalloc_ptr[device]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[device] = p;
  }
  *out = g_noalloc_ptr[device];
  return cudaSuccess;
}

}  // namespace
}  // namespace akv

extern "C" int audiokv_score_noalloc(int device, const audiokv_params* p, const void* q_win, const void* k,
                                     float* scores, audiokv_stream stream) {
  using namespace akv;
  if (!p || !p->seq_len || !q_win || !k || !scores) return AUDIOKV_EINVAL;
  if (device < 0 || device >= kNoAllocMaxDevices) return AUDIOKV_EINVAL;
  if (p->dtype != AUDIOKV_F32 && p->dtype != AUDIOKV_BF16) return AUDIOKV_EINVAL;
  if (p->n_layers < 1 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->n_q_heads % p->n_kv_heads) return AUDIOKV_EINVAL;
  if (p->n_req < 1 || p->n_req > kNoAllocMaxReq || p->window < 1) return AUDIOKV_EINVAL;
  if (p->head_dim != 64 && p->head_dim != 128 && p->head_dim != 256) return AUDIOKV_EUNSUPPORTED;
  if (p->page_size != 0) return AUDIOKV_EUNSUPPORTED;  // contiguous K only
  const int G = p->n_q_heads / p->n_kv_heads;
  const int64_t R = static_cast<int64_t>(p->window) * G;
  if (R > 1024) return AUDIOKV_EUNSUPPORTED;
  if (static_cast<int64_t>(p->n_layers) * p->n_kv_heads > 2048) return AUDIOKV_EUNSUPPORTED;  // as audiokv_score
  const int per16 = p->dtype == AUDIOKV_F32 ? 4 : 8;
  const int64_t strides[] = {p->q_stride_req, p->q_stride_layer, p->q_stride_tok, p->q_stride_head,
                             p->kv_stride_layer, p->kv_stride_tok, p->kv_stride_head};
  for (int64_t s : strides) {
    if (s < 0) return AUDIOKV_EINVAL;
    if (s % per16) return AUDIOKV_EALIGN;
  }
  if ((reinterpret_cast<uintptr_t>(q_win) | reinterpret_cast<uintptr_t>(k)) & 15u) return AUDIOKV_EALIGN;
  static_assert(sizeof(ReqDesc) * kNoAllocMaxReq <= kNoAllocTableBytes, "request table must fit its slot");

  Shape sh{};
  sh.dtype = p->dtype;
  sh.n_layers = p->n_layers;
  sh.n_q_heads = p->n_q_heads;
  sh.n_kv_heads = p->n_kv_heads;
  sh.head_dim = p->head_dim;
  sh.n_req = p->n_req;
  sh.window = p->window;
  sh.group = G;
  sh.heads_per_req = p->n_layers * p->n_kv_heads;
  sh.total_heads = sh.heads_per_req * p->n_req;
  sh.q_stride_layer = p->q_stride_layer;
  sh.q_stride_tok = p->q_stride_tok;
  sh.q_stride_head = p->q_stride_head;
  sh.kv_stride_layer = p->kv_stride_layer;
  sh.kv_stride_tok = p->kv_stride_tok;
  sh.kv_stride_head = p->kv_stride_head;
  sh.softmax_scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf(static_cast<float>(p->head_dim));
  sh.scale_log2e = static_cast<float>(static_cast<double>(sh.softmax_scale) * 1.4426950408889634);

  NoAllocTable table{};
  ReqDesc* reqs = table.r;
  int max_L = 0;
  int64_t score_off = 0;
  for (int r = 0; r < p->n_req; ++r) {
    const int L = p->seq_len[r];
    if (L <= p->window || L > AUDIOKV_MAX_SEQ_LEN) return AUDIOKV_EINVAL;
    const int64_t off = p->kv_req_offset ? p->kv_req_offset[r] : 0;
    if (off < 0) return AUDIOKV_EINVAL;
    if (off % per16) return AUDIOKV_EALIGN;
    const int64_t q_off = p->q_req_offset ? p->q_req_offset[r] : r * p->q_stride_req;
    if (q_off < 0) return AUDIOKV_EINVAL;
    if (q_off % per16) return AUDIOKV_EALIGN;
    reqs[r] = ReqDesc{L, L - p->window, r * sh.heads_per_req, 0, off, q_off, score_off};
    score_off += static_cast<int64_t>(sh.heads_per_req) * (L - p->window);
    max_L = L > max_L ? L : max_L;
  }
  constexpr int kSlabKeys = 512;
  const int n_slab = (max_L + kSlabKeys - 1) / kSlabKeys;
  const size_t need = sizeof(float2) * static_cast<size_t>(sh.total_heads) * n_slab * static_cast<size_t>(R);
  if (need > kNoAllocBytes - kNoAllocTableBytes) return AUDIOKV_EWORKSPACE;  // beyond the fixed scratch

  if (cudaSetDevice(device) != cudaSuccess) return AUDIOKV_ECUDA;
  void* base = nullptr;
  if (noalloc_scratch(device, &base) != cudaSuccess) return AUDIOKV_ECUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  noalloc_table_kernel<<<1, kNoAllocMaxReq, 0, s>>>(table, p->n_req, static_cast<ReqDesc*>(base));
  if (cudaGetLastError() != cudaSuccess) return AUDIOKV_ECUDA;
  int64_t launches = 0;
  Launch ln{s, &launches, nullptr};
  // Sweep 1 writes every statistics entry that sweep 2 reads, so nothing has to start at zero.
  cudaError_t e = launch_score_simt(sh, static_cast<const ReqDesc*>(base), q_win, k, scores,
                                    reinterpret_cast<float2*>(static_cast<unsigned char*>(base) + kNoAllocTableBytes),
                                    n_slab, kSlabKeys, ln);
  return e == cudaSuccess ? AUDIOKV_OK : AUDIOKV_ECUDA;
}
