// Shared declarations of the CUDA side of the AudioKV eviction pass (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <vector>
#include <stdint.h>

#include "../../include/audiokv.h"

namespace akv {

// One request of the ragged batch, as the kernels see it.
struct ReqDesc {
  int32_t L;             // cached tokens
  int32_t P;             // prefix tokens = L - W
  int32_t head_base;     // flat index of the request's first head
  int32_t fft_plan;      // index into the FFT plan table (one per distinct P)
  int64_t kv_offset;     // element offset of the request inside K / V
  int64_t q_offset;      // element offset of the request inside Q
  int64_t score_offset;  // element offset of the request inside a packed score buffer
};

// Shape data common to all kernels; passed by value.
struct Shape {
  int32_t dtype, n_layers, n_q_heads, n_kv_heads, head_dim, n_req, window, group;  // group = G
  int32_t heads_per_req;  // N = n_layers * n_kv_heads
  int32_t total_heads;    // n_req * N
  int64_t q_stride_layer, q_stride_tok, q_stride_head;
  int64_t kv_stride_layer, kv_stride_tok, kv_stride_head;
  float scale_log2e;  // softmax_scale * log2(e): logits are taken to base 2
  float softmax_scale;
  float rho, alpha;
  int32_t transition_bins, base_per_head;
  int32_t smooth_mode, pool_kernel;  // AUDIOKV_SMOOTH_*; window of the pooling modes
  float smooth_kappa;                // cut-off fraction of AUDIOKV_SMOOTH_FIXED_FRACTION
  // paged K / V: page_size 0 = contiguous; page_shift = log2(page_size)
  int32_t page_size, page_shift, n_pages;
  int64_t page_table_stride;
  const int32_t* page_table;  // device [n_req][page_table_stride]
  int* page_status;           // status word that a page id outside the pool is reported to (may be null)
};

// Element offset of token j of request r inside K / V, without the layer and head terms. A page id outside the pool
// is reported through the status word and read as page 0, so that no address leaves the pool.
__device__ __forceinline__ int64_t kv_token_offset(const Shape& sh, const ReqDesc& rq, int r, int j) {
  if (sh.page_size == 0) return rq.kv_offset + static_cast<int64_t>(j) * sh.kv_stride_tok;
  int page = __ldg(sh.page_table + r * sh.page_table_stride + (j >> sh.page_shift));
  if (page < 0 || page >= sh.n_pages) {
    if (sh.page_status) atomicExch(sh.page_status, AUDIOKV_EDEVICE);
    page = 0;
  }
  return ((static_cast<int64_t>(page) << sh.page_shift) + (j & (sh.page_size - 1))) * sh.kv_stride_tok;
}

// Maps a flat head index to (request, layer, kv head). n_req is small: linear search.
__device__ __forceinline__ int find_req(const ReqDesc* __restrict__ reqs, int n_req, int heads_per_req, int u) {
  int r = u / heads_per_req;
  return r < n_req ? r : n_req - 1;
}

// ---- FFT plans -------------------------------------------------------------------------
constexpr int kMaxRadices = 20;

// How one complex transform of length N is carried out (Stockham passes over `radix`).
struct FftSeq {
  int32_t N;
  int32_t n_pass;
  int32_t radix[kMaxRadices];
  int64_t tw_offset;  // float2 index of W_N^t, t in [0, N), inside the table area
};

// Plan for a real sequence of length n (one per distinct prefix length in the batch).
struct FftPlan {
  int32_t n;         // real length
  int32_t packed;    // 1: n even, transform z_m = x_2m + i x_2m+1 of length n/2; 0: length n with zero imaginary part
  int32_t N;         // complex transform length (n/2 or n)
  int32_t bluestein; // 1: N goes through a chirp-z convolution of length M (a product of 2, 3, 5, 7)
  int32_t half;      // bluestein, not packed (odd n): only bins 0 .. (n-1)/2 are computed and fed back, M >= N + (N-1)/2
  int32_t M;         // convolution length (bluestein only)
  int32_t in_smem;   // 1: the work buffer fits in shared memory
  int32_t tabs_smem; // 1: twiddles, post-twiddles and bin positions are staged in shared memory after the buffer
  int32_t g_pass;    // not in_smem: leading passes that run on the global buffer; the rest runs block by block in shared memory
  FftSeq seq;        // passes for length N (direct) or M (bluestein)
  int64_t chirp_offset;   // float2 index of c_j = exp(-i pi j^2 / N), j in [0, N)      (bluestein)
  int64_t filter_offset;  // float2 index of FFT_M of the wrapped conjugate chirp / M    (bluestein)
  int64_t filter2_offset; // half: the same for the inverse direction's wrap (few inputs, all outputs)
  int64_t post_offset;    // float2 index of exp(-2 pi i k / n), k in [0, N/2]           (packed)
  int64_t pos_offset;     // float2 index of an int32 table: slot of bin k after the forward passes (direct)
};


// float2 slots of a shared-memory work buffer of `len` elements: element i sits at i + (i >> 4) (see SkewBuf in sss.cu)
__host__ __device__ inline int sss_padded(int len) { return len + (len >> 4) + 1; }

// SMs of the current device, asked once per device (grids of the bandwidth-bound kernels are sized by it).
inline int device_sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
    cached[dev] = n;
  }
  return cached[dev];
}

// ---- launchers (one per source file) ---------------------------------------------------
// Optional per-kernel timing: an event after every kernel launch of one call.
struct Profiler {
  static constexpr int kMax = 32;
  bool on = false;
  int n = 0;                 // events recorded in the current call (event 0 = start of the call)
  cudaEvent_t ev[kMax] = {};
  const char* name[kMax] = {};
};

struct Launch {
  cudaStream_t stream;
  int64_t* launch_counter;
  Profiler* prof;
  // Counts one kernel launch and, when profiling, records the event that ends it.
  void done(const char* kernel_name) const {
    *launch_counter += 1;
    if (prof && prof->on && prof->n < Profiler::kMax) {
      cudaEventRecord(prof->ev[prof->n], stream);
      prof->name[prof->n] = kernel_name;
      prof->n += 1;
    }
  }
};

// Programmatic dependent launch: a kernel launched with launch_chained may be set up on the SMs while the
// kernel before it on the stream is still draining. Such a kernel calls chain_wait() before it touches global
// memory (it returns once every earlier kernel has finished and its writes are visible), and every kernel
// calls chain_release() at its start so that its successor may be brought in early.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                           Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// score_simt.cu: fp32-FMA scoring for any dtype. stats_ws: float2 [total_heads][n_slab][rows].
cudaError_t launch_score_simt(const Shape& sh, const ReqDesc* d_reqs, const void* q, const void* k, float* scores,
                              float2* stats_ws, int n_slab, int slab_keys, Launch ln);

// One run of work of the tensor-core scoring kernel: consecutive key tiles of one head (of one chunk of its window
// rows) that one CTA processes. The schedule of each sweep is a table of these, built on the host in processing
// order, so that no role of the kernel divides to find its work.
struct ScoreUnit {
  int32_t u, r, l, h;              // flat head, request, layer, KV head
  int32_t part, kt0, n_tiles, P;   // statistics slot of the run (sweep 1), first key, K tiles of 128 keys, prefix length
  int64_t score_base;              // element offset of the head's scores in a packed score buffer
  int32_t head_parts;              // runs sweep 1 made of this head (statistics slots that sweep 2 merges)
  int32_t w0, wn;                  // window rows [w0, w0 + wn) of the head: the query rows this run works on
  int32_t qid;                     // u * (window chunks per head) + chunk: changes whenever another Q tile is needed
};

// One launch of the two sweeps: the heads it covers and where its runs lie in the device tables. CTA c of sweep s
// takes the runs cta[c] .. cta[c + 1] - 1, cta = the grid[s] + 1 entries at cta_off[s] of the CTA table.
struct ScoreSchedule {
  int32_t whole_requests;          // 1: all heads of requests [r_begin, r_end); 0: heads [head_begin, head_end) of request 0
  int32_t r_begin, r_end;
  int32_t head_begin, head_end;
  int32_t unit_off[2], cta_off[2], grid[2];
};

// CTAs the tiles of a launch are dealt out over (the SM count of the part this library is built for; fewer when there
// are fewer tiles). A device with more SMs leaves some idle, one with fewer runs the CTAs in turn: no CTA waits for another.
constexpr int kScoreCtas = 148;

// Window rows per run of the tensor-core scoring: the largest share of the window whose W_c * G query rows fit the
// kernel (256 rows; 128 at head_dim 256, where only a 128-row Q tile leaves room for two K stages), 0 if G alone
// does not fit. A head whose W * G is larger is scored in ceil(W / W_c) chunks of window rows.
int score_window_chunk(const Shape& sh);
// Statistics entries sweep 1 of the tensor-core scoring writes per part of a head (its epilogue groups and sets).
int score_stat_sets();
// Requests whose tensor maps travel with one launch (8 for a small batch, 120 for a long one).
int score_map_chunk(int n_req);

// score_umma.cu: bf16 scoring on the tcgen05 tensor cores. score_umma_takes says whether the shape fits the kernel;
// the launcher returns cudaErrorNotSupported when the strides cannot be described to the copy engine, and the caller
// then scores with launch_score_simt. h_reqs: host copy of the request table (the tensor maps are encoded on the host).
bool score_umma_takes(const Shape& sh);
// Limit, in SM clock cycles, of the waits on mbarriers inside the tensor-core scoring kernels (about one second by
// default). A wait that runs out stops its CTA and the kernel reports AUDIOKV_ETIMEOUT. cycles <= 0 restores the default.
void set_score_wait_cycles(long long cycles);
long long score_wait_cycles();
// The encoded tensor maps of the last call, kept by the context: encoding a few hundred maps costs more host time than
// the kernels take on a short cache, and a serving loop calls with the same buffers and the same plan again and again.
struct ScoreMapCache {
  const void* q = nullptr;
  const void* k = nullptr;
  uint64_t plan_id = 0;   // changes whenever the plan is rebuilt
  int page_size = -1;
  std::vector<unsigned char> packs;   // one argument pack per run of requests
  std::vector<unsigned char> encoded; // which of them hold maps of these buffers
};
// d_units / d_cta: device tables of runs and per-CTA offsets (both sweeps of every schedule). scheds: host.
// head_end < 0: every whole-request schedule in turn; else the schedule made for heads [head_begin, head_end).
// stats_ws: float2 [total heads][max_parts][score_stat_sets()][W * G].
// beside: the kernel launched just before on the stream is the library's own budget kernel (ordinary launch, calls
// chain_release at once): the first sweep then runs beside it instead of after it.
cudaError_t launch_score_umma(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* d_units, const int32_t* d_cta,
                              const ScoreSchedule* scheds, int n_sched, const void* q, const void* k, float* scores,
                              float2* stats_ws, int max_parts, int* status, Launch ln, int head_begin = 0,
                              int head_end = -1, ScoreMapCache* cache = nullptr, uint64_t plan_id = 0, bool beside = false);

// sss.cu
cudaError_t launch_fft_tables(int n_plans, float2* d_tables, const FftPlan* d_plans, Launch ln);
// order: n_order head indices (or -1); block b takes entries b, b + grid, ... ; a null order stands for the n_order heads
// first_head, first_head + 1, ... . smoothed may be null when budgets, cu_kept and kept_idx are given: the kernel then goes on to the
// top-k selection of each head from the smoothed scores it holds on chip (step 4a of the pass).
cudaError_t launch_sss(const Shape& sh, const ReqDesc* d_reqs, const FftPlan* d_plans, const float2* d_tables,
                       const float* scores, float* smoothed, int32_t* kstar, float2* scratch,
                       int64_t scratch_per_block, int grid, size_t smem_bytes, const int32_t* order, int n_order,
                       int first_head, const int32_t* budgets, const int32_t* cu_kept, int32_t* kept_idx, int* status,
                       Launch ln);

// allocate.cu (h_total_budget: host array [n_req])
cudaError_t launch_allocate(const Shape& sh, const ReqDesc* d_reqs, const float* head_scores,
                            const int64_t* h_total_budget, int32_t* budgets, int32_t* cu_kept, int* status,
                            Launch ln);

// given: device int32 [total heads], budgets chosen by the caller; budgets: their checked copy; cu_kept: prefix sums.
cudaError_t launch_budget_prefix(const Shape& sh, const ReqDesc* d_reqs, const int32_t* given, int32_t* budgets,
                                 int32_t* cu_kept, int* status, Launch ln);

// select_gather.cu
cudaError_t launch_select(const Shape& sh, const ReqDesc* d_reqs, const float* smoothed, const int32_t* budgets,
                          const int32_t* cu_kept, int32_t* kept_idx, int max_P, int* status, Launch ln);
// head_begin / head_end: the rows of heads [head_begin, head_end) only (0, total heads = everything).
cudaError_t launch_gather(const Shape& sh, const ReqDesc* d_reqs, const int32_t* cu_kept, const int32_t* kept_idx,
                          const void* k, const void* v, void* k_out, void* v_out, int head_begin, int head_end,
                          Launch ln);

// hit_score.cu: offline head score. counts: int32 [n_heads] (cleared here, then the hit totals).
cudaError_t launch_hit_score(const float* attn, int n_steps, int n_heads, int64_t row_stride, const int32_t* row_len,
                             const int32_t* span, int top_k, int32_t* counts, float* s_hit, int* status, Launch ln);

// spread.cu: histogram of the kept prefix tokens over n_bins stretches of each request's prefix (hist int32
// [n_req][n_bins], cleared here) and its summaries (stats fp32 [n_req][2]: balance, peak).
cudaError_t launch_selection_spread(const Shape& sh, const ReqDesc* d_reqs, const int32_t* kept_idx,
                                    const int32_t* cu_kept, int n_bins, int32_t* hist, float* stats, int* status,
                                    Launch ln);

}  // namespace akv
