// C boundary of the AudioKV eviction pass: argument checks, the per-shape plan (request
// table, FFT plans and tables, workspace layout) and the launch sequence of each entry point.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <unordered_map>
#include <vector>

#include "common.cuh"

using namespace akv;

namespace {

constexpr size_t kAlign = 256;
constexpr int kSssSmemComplex = 25600;  // 200 KB of float2: the largest work buffer kept in shared memory
constexpr int kSlabKeys = 256;          // keys per slab of the softmax statistics (two K tiles of the tensor-core kernel)
constexpr int kMaxRows = 1024;          // W * G
constexpr int kMaxHeadsPerReq = 2048;
constexpr int kHostChunks = 8;          // the host-buffer call evicts one request in at most this many runs of layers

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {  // byte offsets inside the workspace
  size_t status, reqs, plans, tables, units, ctas, order, stats, fft_scratch, scores, kstar, aux, end;
};

struct Plan {
  bool valid = false;
  audiokv_params p{};
  std::vector<int32_t> seq_len;
  std::vector<int64_t> kv_off, q_off;
  Shape sh{};
  std::vector<ReqDesc> reqs;
  std::vector<FftPlan> fft;
  std::vector<ScoreUnit> units;          // runs of the tensor-core scoring: both sweeps of every schedule
  std::vector<int32_t> score_ctas;       // per-CTA run offsets of every (schedule, sweep)
  std::vector<ScoreSchedule> schedules;  // one per run of requests, plus one per chunk of layers of a single request
  int score_parts = 1;                   // statistics slots per head of the tensor-core scoring
  std::vector<int32_t> sss_order;  // heads in the order the smoothing blocks take them (see build_plan); -1 = none
  int64_t table_len = 0;        // float2 elements
  int64_t scores_len = 0;
  int max_L = 0, max_P = 0;
  int n_slab = 0;
  int sss_grid = 0;
  size_t sss_smem = 0;
  int64_t scratch_per_block = 0;  // float2 elements
  Layout lay{};
};

// Host arrays of the per-head problem that audiokv_reevict derives from its arguments.
struct ReevictArrays {
  std::vector<int32_t> len;
  std::vector<int64_t> kv_off, q_off, budget;
};

}  // namespace

struct audiokv_ctx {
  int device = 0;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  Plan plan;
  bool plan_uploaded = false;
  uint64_t plan_id = 0;      // counts plan rebuilds
  ScoreMapCache score_maps;
  cudaEvent_t plan_ready = nullptr;
  cudaStream_t side = nullptr;            // audiokv_evict runs the allocation here, beside the scoring
  cudaEvent_t fork = nullptr, join = nullptr;
  // audiokv_evict_host: copies in on `side`, kernels on the caller's stream, copies out on `out`, chunk by chunk
  static constexpr int kMaxChunks = kHostChunks;
  cudaStream_t out = nullptr;
  cudaEvent_t chunk_in[kMaxChunks] = {}, chunk_done[kMaxChunks] = {}, copies_out = nullptr;
  int64_t launches = 0;
  int score_path = 0;  // route of the last scoring: 0 none yet, 1 tensor cores, 2 fp32 FMA
  Profiler prof;
  std::string cuda_error;
  ReevictArrays re;  // audiokv_reevict: the per-head problem it hands to the eviction pass
};

namespace {

int esize(int dtype) { return dtype == AUDIOKV_F32 ? 4 : 2; }

int check_params(const audiokv_params* p) {
  if (!p || !p->seq_len) return AUDIOKV_EINVAL;
  if (p->dtype != AUDIOKV_F32 && p->dtype != AUDIOKV_BF16) return AUDIOKV_EINVAL;
  if (p->n_layers < 1 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->n_q_heads % p->n_kv_heads) return AUDIOKV_EINVAL;
  if (p->n_req < 1 || p->n_req > AUDIOKV_MAX_REQ || p->window < 1) return AUDIOKV_EINVAL;
  if (!(p->rho > 0.f && p->rho <= 1.f) || !(p->alpha >= 0.f && p->alpha <= 1.f)) return AUDIOKV_EINVAL;
  if (p->transition_bins < 0 || p->base_per_head < 0) return AUDIOKV_EINVAL;
  if (p->smooth_mode < AUDIOKV_SMOOTH_SSS || p->smooth_mode > AUDIOKV_SMOOTH_MAX_POOL) return AUDIOKV_EINVAL;
  if (p->smooth_mode == AUDIOKV_SMOOTH_FIXED_FRACTION && !(p->smooth_kappa >= 0.f && p->smooth_kappa <= 1.f))
    return AUDIOKV_EINVAL;
  if (p->smooth_mode >= AUDIOKV_SMOOTH_AVG_POOL && (p->pool_kernel < 1 || p->pool_kernel > 1023 || p->pool_kernel % 2 == 0))
    return AUDIOKV_EINVAL;
  for (int r = 0; r < p->n_req; ++r) {
    if (p->seq_len[r] <= p->window || p->seq_len[r] > AUDIOKV_MAX_SEQ_LEN) return AUDIOKV_EINVAL;
    if (p->kv_req_offset && p->kv_req_offset[r] < 0) return AUDIOKV_EINVAL;
    if (p->q_req_offset && p->q_req_offset[r] < 0) return AUDIOKV_EINVAL;
  }
  if (p->head_dim != 64 && p->head_dim != 128 && p->head_dim != 256) return AUDIOKV_EUNSUPPORTED;
  const int64_t rows = static_cast<int64_t>(p->window) * (p->n_q_heads / p->n_kv_heads);
  if (rows > kMaxRows) return AUDIOKV_EUNSUPPORTED;
  if (static_cast<int64_t>(p->n_layers) * p->n_kv_heads > kMaxHeadsPerReq) return AUDIOKV_EUNSUPPORTED;
  const int per16 = 16 / esize(p->dtype);
  const int64_t strides[] = {p->q_stride_req, p->q_stride_layer, p->q_stride_tok, p->q_stride_head,
                             p->kv_stride_layer, p->kv_stride_tok, p->kv_stride_head};
  for (int64_t s : strides) {
    if (s < 0) return AUDIOKV_EINVAL;
    if (s % per16) return AUDIOKV_EALIGN;
  }
  if (p->page_size != 0) {
    if (p->page_size != 16 && p->page_size != 32 && p->page_size != 64 && p->page_size != 128) return AUDIOKV_EUNSUPPORTED;
    if (p->n_pages < 1 || !p->page_table || p->kv_stride_tok < 1) return AUDIOKV_EINVAL;
    if (static_cast<int64_t>(p->n_pages) * p->page_size > 0x7fffffffLL) return AUDIOKV_EUNSUPPORTED;
    for (int r = 0; r < p->n_req; ++r)
      if ((p->seq_len[r] + p->page_size - 1) / p->page_size > p->page_table_stride) return AUDIOKV_EINVAL;
  }
  for (int r = 0; r < p->n_req; ++r) {
    if (p->kv_req_offset && p->kv_req_offset[r] % per16) return AUDIOKV_EALIGN;
    if (p->q_req_offset && p->q_req_offset[r] % per16) return AUDIOKV_EALIGN;
  }
  return AUDIOKV_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool same_plan(const Plan& pl, const audiokv_params* p) {
  if (!pl.valid) return false;
  const audiokv_params& a = pl.p;
  if (a.dtype != p->dtype || a.n_layers != p->n_layers || a.n_q_heads != p->n_q_heads ||
      a.n_kv_heads != p->n_kv_heads || a.head_dim != p->head_dim || a.n_req != p->n_req || a.window != p->window ||
      a.q_stride_layer != p->q_stride_layer ||
      a.q_stride_tok != p->q_stride_tok || a.q_stride_head != p->q_stride_head ||
      a.kv_stride_layer != p->kv_stride_layer || a.kv_stride_tok != p->kv_stride_tok ||
      a.kv_stride_head != p->kv_stride_head || a.softmax_scale != p->softmax_scale || a.rho != p->rho ||
      a.alpha != p->alpha || a.transition_bins != p->transition_bins || a.base_per_head != p->base_per_head ||
      a.smooth_mode != p->smooth_mode || a.smooth_kappa != p->smooth_kappa || a.pool_kernel != p->pool_kernel ||
      a.page_size != p->page_size || a.n_pages != p->n_pages || a.page_table_stride != p->page_table_stride)
    return false;
  for (int r = 0; r < p->n_req; ++r) {
    if (pl.seq_len[r] != p->seq_len[r]) return false;
    if (pl.kv_off[r] != (p->kv_req_offset ? p->kv_req_offset[r] : 0)) return false;
    if (pl.q_off[r] != (p->q_req_offset ? p->q_req_offset[r] : r * p->q_stride_req)) return false;
  }
  return true;
}

// Radix sequence for a complex length N: primes 11..127 first (descending), then 7, 5, 3, 4s, 2.
// Returns false when N has a prime factor above 127.
bool factor_len(int N, FftSeq* sq) {
  sq->N = N;
  sq->n_pass = 0;
  int rest = N, twos = 0;
  while (rest % 2 == 0) {
    rest /= 2;
    ++twos;
  }
  std::vector<int> odd;
  for (int q = 3; q <= 127 && rest > 1; q += 2)
    while (rest % q == 0) {
      odd.push_back(q);
      rest /= q;
    }
  if (rest != 1) return false;
  std::vector<int> seq;
  for (auto it = odd.rbegin(); it != odd.rend(); ++it) seq.push_back(*it);
  for (int i = 0; i < twos / 2; ++i) seq.push_back(4);
  if (twos % 2) seq.push_back(2);
  if (seq.size() > static_cast<size_t>(kMaxRadices)) return false;
  for (size_t i = 0; i < seq.size(); ++i) sq->radix[i] = seq[i];
  sq->n_pass = static_cast<int>(seq.size());
  return true;
}

// float2 slots of shared memory a plan's block needs: the work buffer, and with tables N (W_N) + N/2 + 1 (post) + N/4 + 1 (positions)
int sss_smem_complex(const FftPlan& fp, bool with_tables) {
  const int len = sss_padded(fp.bluestein ? fp.M : fp.N);
  return len + (with_tables ? fp.N + fp.N / 2 + 1 + fp.N / 4 + 1 : 0);
}

void build_fft_plan(int n, FftPlan* fp, int64_t* table_len) {
  memset(fp, 0, sizeof(*fp));
  fp->n = n;
  fp->packed = (n % 2 == 0) ? 1 : 0;
  fp->N = fp->packed ? n / 2 : n;
  const int N = fp->N;
  int buf_len = N;
  if (factor_len(N, &fp->seq)) {
    fp->bluestein = 0;
    fp->M = 0;
  } else {
    fp->bluestein = 1;
    // An odd real length is transformed at full complex length N = n, but only bins 0 .. (n-1)/2 are wanted (the rest
    // mirror them) and only those go back into the inverse: differences between input and output indices then span
    // N + (N-1)/2 values instead of 2N - 1, and the convolution may be that much shorter.
    fp->half = fp->packed ? 0 : 1;
    const int64_t need = fp->half ? static_cast<int64_t>(N) + (N - 1) / 2 : 2LL * N - 1;
    // convolution length: the smallest 2^a 3^b 5^c 7^d (a >= 2) that holds `need` points; close to it
    // instead of up to twice that for a power of two, which also keeps more transforms in shared memory
    int M = 0;
    for (int64_t p7 = 1; p7 < 4LL * N; p7 *= 7)
      for (int64_t p5 = p7; p5 < 4LL * N; p5 *= 5)
        for (int64_t p3 = p5; p3 < 4LL * N; p3 *= 3)
          for (int64_t p2 = p3 * 4; p2 < 8LL * N; p2 *= 2)
            if (p2 >= need) {
              if (M == 0 || p2 < M) M = static_cast<int>(p2);
              break;
            }
    fp->M = M;
    factor_len(M, &fp->seq);
    buf_len = M;
  }
  fp->in_smem = sss_padded(buf_len) <= kSssSmemComplex ? 1 : 0;
  fp->g_pass = 0;
  if (!fp->in_smem) {
    // leading passes on the global buffer until a block and its twiddles (padded(len) + len slots) fit on chip
    int len = buf_len;
    while (fp->g_pass < fp->seq.n_pass && sss_padded(len) + len > kSssSmemComplex) len /= fp->seq.radix[fp->g_pass++];
  }
  // a direct transform also keeps its tables on chip when buffer + W_N + post-twiddles + uint16 positions fit
  fp->tabs_smem = (!fp->bluestein && fp->in_smem && N < 65536 && sss_smem_complex(*fp, true) <= kSssSmemComplex) ? 1 : 0;
  fp->seq.tw_offset = *table_len;
  *table_len += fp->seq.N;
  if (fp->packed) {
    fp->post_offset = *table_len;
    *table_len += N / 2 + 1;
  }
  if (!fp->bluestein) {
    fp->pos_offset = *table_len;
    *table_len += (N + 1) / 2;  // N int32 entries
  }
  if (fp->bluestein) {
    fp->chirp_offset = *table_len;
    *table_len += N;
    fp->filter_offset = *table_len;
    *table_len += fp->M;
    if (fp->half) {
      fp->filter2_offset = *table_len;
      *table_len += fp->M;
    }
  }
}

int host_chunks(int n_layers) { return n_layers < kHostChunks ? n_layers : kHostChunks; }
int host_chunk_layer(int n_layers, int c) { return static_cast<int>(static_cast<int64_t>(n_layers) * c / host_chunks(n_layers)); }

// Schedules of the tensor-core scoring. A schedule covers a set of heads; the key tiles of those heads, in the order
// the sweep walks them, are dealt out evenly over the CTAs, CTA c taking tiles [c T / grid, (c + 1) T / grid): a few
// runs of consecutive tiles of one head. Sweep 1 walks the heads in order over all L keys (the runs of a head number
// its statistics slots); sweep 2 walks them backwards over the prefix keys (the heads sweep 1 touched last are the
// ones still in L2).
void build_score_schedules(const audiokv_params* p, Plan* pl) {
  const Shape& sh = pl->sh;
  pl->units.clear();
  pl->score_ctas.clear();
  pl->schedules.clear();
  pl->score_parts = 1;
  if (!score_umma_takes(sh)) return;
  // a head whose W * G query rows exceed the kernel's Q tile is scored in chunks of window rows (runs of their own)
  const int w_chunk = score_window_chunk(sh);
  const int n_wchunks = (p->window + w_chunk - 1) / w_chunk;
  std::vector<int32_t> parts_of(static_cast<size_t>(sh.total_heads) * n_wchunks, 0);
  auto add = [&](bool whole, int r_begin, int r_end, int head_begin, int head_end) {
    ScoreSchedule sc{};
    sc.whole_requests = whole ? 1 : 0;
    sc.r_begin = r_begin;
    sc.r_end = r_end;
    sc.head_begin = head_begin;
    sc.head_end = head_end;
    struct Q {
      int u, r, hr, ch;
    };
    std::vector<Q> qs;  // the (head, window chunk) pairs of this schedule, in sweep-1 order
    for (int r = r_begin; r < r_end; ++r)
      for (int hr = whole ? 0 : head_begin; hr < (whole ? sh.heads_per_req : head_end); ++hr)
        for (int ch = 0; ch < n_wchunks; ++ch) qs.push_back(Q{pl->reqs[r].head_base + hr, r, hr, ch});
    for (int sweep = 1; sweep <= 2; ++sweep) {
      if (sweep == 2) std::reverse(qs.begin(), qs.end());
      int64_t total = 0;
      for (const Q& x : qs) {
        const int range = sweep == 1 ? pl->reqs[x.r].L : pl->reqs[x.r].P;
        total += (range + 127) / 128;
      }
      const int grid = static_cast<int>(total < kScoreCtas ? total : kScoreCtas);
      sc.unit_off[sweep - 1] = static_cast<int32_t>(pl->units.size());
      sc.cta_off[sweep - 1] = static_cast<int32_t>(pl->score_ctas.size());
      sc.grid[sweep - 1] = grid;
      const size_t first = pl->units.size();
      int64_t tile = 0;  // tiles before the current head in the sweep's sequence
      int c = 0;         // CTA whose range holds the next tile
      pl->score_ctas.push_back(0);
      for (const Q& x : qs) {
        const ReqDesc& d = pl->reqs[x.r];
        const int range = sweep == 1 ? d.L : d.P;
        const int n_tiles = (range + 127) / 128;
        int t = 0, part = 0;
        while (t < n_tiles) {
          // the CTA that owns tile `tile + t`, and how far its range reaches into this head
          while (c + 1 < grid && (static_cast<int64_t>(c + 1) * total) / grid <= tile + t) {
            ++c;
            pl->score_ctas.push_back(static_cast<int32_t>(pl->units.size() - first));
          }
          const int64_t c_end = (static_cast<int64_t>(c + 1) * total) / grid;
          const int take = static_cast<int>(std::min<int64_t>(n_tiles - t, c_end - (tile + t)));
          ScoreUnit un{};
          un.u = x.u;
          un.r = x.r;
          un.l = x.hr / p->n_kv_heads;
          un.h = x.hr % p->n_kv_heads;
          un.part = part++;
          un.kt0 = t * 128;
          un.n_tiles = take;
          un.P = d.P;
          un.score_base = d.score_offset + static_cast<int64_t>(x.hr) * d.P;
          un.w0 = x.ch * w_chunk;
          un.wn = p->window - un.w0 < w_chunk ? p->window - un.w0 : w_chunk;
          un.qid = x.u * n_wchunks + x.ch;
          un.head_parts = 0;  // set below
          pl->units.push_back(un);
          t += take;
        }
        if (sweep == 1) {
          parts_of[static_cast<size_t>(x.u) * n_wchunks + x.ch] = part;
          pl->score_parts = part > pl->score_parts ? part : pl->score_parts;
        }
        tile += n_tiles;
      }
      while (static_cast<int>(pl->score_ctas.size()) - sc.cta_off[sweep - 1] < grid + 1)
        pl->score_ctas.push_back(static_cast<int32_t>(pl->units.size() - first));
      for (size_t i = first; i < pl->units.size(); ++i) pl->units[i].head_parts = parts_of[pl->units[i].qid];
    }
    pl->schedules.push_back(sc);
  };
  const int cap = score_map_chunk(p->n_req);
  for (int r0 = 0; r0 < p->n_req; r0 += cap) add(true, r0, r0 + cap < p->n_req ? r0 + cap : p->n_req, 0, 0);
  if (p->n_req == 1 && p->n_layers > 1) {
    // the host-buffer call evicts one request in chunks of layers
    const int n_chunks = host_chunks(p->n_layers);
    for (int c = 0; c < n_chunks; ++c)
      add(false, 0, 1, host_chunk_layer(p->n_layers, c) * p->n_kv_heads, host_chunk_layer(p->n_layers, c + 1) * p->n_kv_heads);
  }
}

int build_plan(const audiokv_params* p, Plan* pl) {
  int rc = check_params(p);
  if (rc) return rc;
  pl->valid = false;
  pl->p = *p;
  pl->seq_len.assign(p->seq_len, p->seq_len + p->n_req);
  pl->kv_off.assign(p->n_req, 0);
  if (p->kv_req_offset) pl->kv_off.assign(p->kv_req_offset, p->kv_req_offset + p->n_req);
  pl->q_off.resize(p->n_req);
  for (int r = 0; r < p->n_req; ++r) pl->q_off[r] = p->q_req_offset ? p->q_req_offset[r] : r * p->q_stride_req;
  pl->p.seq_len = nullptr;
  pl->p.kv_req_offset = nullptr;
  pl->p.q_req_offset = nullptr;
  pl->p.page_table = nullptr;

  Shape& sh = pl->sh;
  sh.dtype = p->dtype;
  sh.n_layers = p->n_layers;
  sh.n_q_heads = p->n_q_heads;
  sh.n_kv_heads = p->n_kv_heads;
  sh.head_dim = p->head_dim;
  sh.n_req = p->n_req;
  sh.window = p->window;
  sh.group = p->n_q_heads / p->n_kv_heads;
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
  sh.rho = p->rho;
  sh.alpha = p->alpha;
  sh.transition_bins = p->transition_bins;
  sh.base_per_head = p->base_per_head;
  sh.smooth_mode = p->smooth_mode;
  sh.smooth_kappa = p->smooth_kappa;
  sh.pool_kernel = p->pool_kernel;
  sh.page_size = p->page_size;
  sh.page_shift = 0;
  while (p->page_size && (1 << sh.page_shift) < p->page_size) ++sh.page_shift;
  sh.n_pages = p->n_pages;
  sh.page_table_stride = p->page_table_stride;
  sh.page_table = nullptr;  // set per call, with the status word
  sh.page_status = nullptr;

  pl->reqs.assign(p->n_req, ReqDesc{});
  pl->fft.clear();
  pl->table_len = 0;
  pl->scores_len = 0;
  pl->max_L = pl->max_P = 0;
  std::unordered_map<int, int> plan_of;  // prefix length -> index into pl->fft
  for (int r = 0; r < p->n_req; ++r) {
    ReqDesc& d = pl->reqs[r];
    d.L = p->seq_len[r];
    d.P = d.L - p->window;
    d.head_base = r * sh.heads_per_req;
    d.kv_offset = pl->kv_off[r];
    d.q_offset = pl->q_off[r];
    d.score_offset = pl->scores_len;
    pl->scores_len += static_cast<int64_t>(sh.heads_per_req) * d.P;
    pl->max_L = d.L > pl->max_L ? d.L : pl->max_L;
    pl->max_P = d.P > pl->max_P ? d.P : pl->max_P;
    auto it = plan_of.find(d.P);
    if (it == plan_of.end()) {
      FftPlan fp;
      build_fft_plan(d.P, &fp, &pl->table_len);
      pl->fft.push_back(fp);
      it = plan_of.emplace(d.P, static_cast<int>(pl->fft.size()) - 1).first;
    }
    d.fft_plan = it->second;
  }
  pl->n_slab = (pl->max_L + kSlabKeys - 1) / kSlabKeys;
  build_score_schedules(p, pl);
  // one block per head at a time, as many blocks as the planning SM count (the plan, and with it the workspace size,
  // does not depend on the device)
  pl->sss_grid = sh.total_heads < kScoreCtas ? sh.total_heads : kScoreCtas;
  {
    // Block b of the smoothing kernel takes entries b, b + grid, b + 2 grid, ... of this list. Heads are sorted by an
    // estimate of their transform's cost and dealt out in a snake (left to right, then right to left), so that
    // a ragged batch with a few expensive lengths (chirp-z in global scratch) does not leave them to one block.
    auto cost = [&](int u) -> double {
      const FftPlan& fp = pl->fft[pl->reqs[u / sh.heads_per_req].fft_plan];
      const double len = fp.bluestein ? fp.M : fp.N;
      double c = len * (fp.bluestein ? 4.0 : 1.0) * (fp.in_smem ? 1.0 : 6.0);
      for (int i = 0; i < fp.seq.n_pass; ++i)
        if (fp.seq.radix[i] > 19) c += static_cast<double>(fp.seq.N) * fp.seq.radix[i] / 8.0;  // O(p N) prime pass
      return c;
    };
    std::vector<int32_t> by_cost(sh.total_heads);
    for (int u = 0; u < sh.total_heads; ++u) by_cost[u] = u;
    std::stable_sort(by_cost.begin(), by_cost.end(), [&](int a, int b) { return cost(a) > cost(b); });
    const int g = pl->sss_grid, tiers = (sh.total_heads + g - 1) / g;
    pl->sss_order.assign(static_cast<size_t>(tiers) * g, -1);
    for (int i = 0; i < sh.total_heads; ++i) {
      const int tier = i / g, j = i - tier * g;
      pl->sss_order[static_cast<size_t>(tier) * g + ((tier & 1) ? g - 1 - j : j)] = by_cost[i];
    }
  }
  int smem_c = 2;
  pl->scratch_per_block = 0;
  for (const FftPlan& fp : pl->fft) {
    const int len = fp.bluestein ? fp.M : fp.N;
    if (fp.in_smem) {
      const int need = sss_smem_complex(fp, fp.tabs_smem != 0);
      smem_c = need > smem_c ? need : smem_c;
    }
    else {
      pl->scratch_per_block = len > pl->scratch_per_block ? len : pl->scratch_per_block;
      int blk = len;
      for (int i = 0; i < fp.g_pass; ++i) blk /= fp.seq.radix[i];
      const int need = sss_padded(blk) + blk;
      smem_c = need > smem_c ? need : smem_c;
    }
  }
  pl->sss_smem = static_cast<size_t>(smem_c) * sizeof(float2);

  Layout& L = pl->lay;
  size_t off = 0;
  L.status = off;      off = align_up(off + 64);
  L.reqs = off;        off = align_up(off + sizeof(ReqDesc) * pl->reqs.size());
  L.plans = off;       off = align_up(off + sizeof(FftPlan) * pl->fft.size());
  L.tables = off;      off = align_up(off + sizeof(float2) * static_cast<size_t>(pl->table_len));
  L.units = off;       off = align_up(off + sizeof(ScoreUnit) * pl->units.size());
  L.ctas = off;        off = align_up(off + sizeof(int32_t) * pl->score_ctas.size());
  L.order = off;       off = align_up(off + sizeof(int32_t) * pl->sss_order.size());
  {
    // softmax statistics: [head][slab][row] for the FMA kernels, [head][part][group][row] for the tensor-core ones
    const size_t slots = std::max<size_t>(pl->n_slab, static_cast<size_t>(pl->score_parts) * score_stat_sets());
    L.stats = off;     off = align_up(off + sizeof(float2) * static_cast<size_t>(sh.total_heads) * slots * sh.window * sh.group);
  }
  L.fft_scratch = off; off = align_up(off + sizeof(float2) * static_cast<size_t>(pl->scratch_per_block) * pl->sss_grid);
  L.scores = off;      off = align_up(off + sizeof(float) * static_cast<size_t>(pl->scores_len));
  L.kstar = off;       off = align_up(off + sizeof(int32_t) * static_cast<size_t>(sh.total_heads));
  L.aux = off;         off = align_up(off + 2 * sizeof(int32_t) * static_cast<size_t>(sh.total_heads));  // audiokv_reevict
  L.end = off;
  pl->valid = true;
  return AUDIOKV_OK;
}

int cuda_fail(audiokv_ctx* ctx, cudaError_t e) {
  ctx->cuda_error = cudaGetErrorString(e);
  return AUDIOKV_ECUDA;
}

// Makes ctx->plan match p and its tables resident on the device (stream-ordered).
int prepare(audiokv_ctx* ctx, const audiokv_params* p, cudaStream_t stream) {
  if (!ctx) return AUDIOKV_EINVAL;
  cudaError_t e = cudaSetDevice(ctx->device);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if (!same_plan(ctx->plan, p)) {
    int rc = build_plan(p, &ctx->plan);
    ctx->plan_id += 1;
    if (rc) return rc;
    ctx->plan_uploaded = false;
  }
  Plan& pl = ctx->plan;
  if (pl.lay.end > ctx->ws_bytes) return AUDIOKV_EWORKSPACE;
  pl.sh.page_table = p->page_size ? p->page_table : nullptr;  // device data of this call, not part of the plan
  pl.sh.page_status = reinterpret_cast<int*>(ctx->ws + pl.lay.status);
  if (!ctx->plan_uploaded) {
    // A new plan goes up with copies from pageable memory, which a stream capture cannot hold: the first call with
    // a given shape has to run outside capture (later ones add nothing but kernels and may be captured).
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if ((e = cudaStreamIsCapturing(stream, &cap)) != cudaSuccess) return cuda_fail(ctx, e);
    if (cap != cudaStreamCaptureStatusNone) {
      ctx->cuda_error = "the plan of these params is not on the device yet: make one call outside stream capture first";
      return AUDIOKV_ECUDA;
    }
    // earlier calls on other streams may still read the old tables
    if ((e = cudaStreamWaitEvent(stream, ctx->plan_ready, 0)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaMemsetAsync(ctx->ws + pl.lay.status, 0, 64, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaMemcpyAsync(ctx->ws + pl.lay.reqs, pl.reqs.data(), sizeof(ReqDesc) * pl.reqs.size(),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess)
      return cuda_fail(ctx, e);
    if ((e = cudaMemcpyAsync(ctx->ws + pl.lay.plans, pl.fft.data(), sizeof(FftPlan) * pl.fft.size(),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess)
      return cuda_fail(ctx, e);
    if (!pl.units.empty() &&
        ((e = cudaMemcpyAsync(ctx->ws + pl.lay.units, pl.units.data(), sizeof(ScoreUnit) * pl.units.size(),
                              cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
         (e = cudaMemcpyAsync(ctx->ws + pl.lay.ctas, pl.score_ctas.data(), sizeof(int32_t) * pl.score_ctas.size(),
                              cudaMemcpyHostToDevice, stream)) != cudaSuccess))
      return cuda_fail(ctx, e);
    if ((e = cudaMemcpyAsync(ctx->ws + pl.lay.order, pl.sss_order.data(), sizeof(int32_t) * pl.sss_order.size(),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess)
      return cuda_fail(ctx, e);
    Launch ln{stream, &ctx->launches, &ctx->prof};
    e = launch_fft_tables(static_cast<int>(pl.fft.size()), reinterpret_cast<float2*>(ctx->ws + pl.lay.tables),
                          reinterpret_cast<const FftPlan*>(ctx->ws + pl.lay.plans), ln);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    // The host waits until the plan is resident (once per shape): calls that follow, on any stream or inside a
    // capture, then need no ordering against the upload.
    if ((e = cudaEventRecord(ctx->plan_ready, stream)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaEventSynchronize(ctx->plan_ready)) != cudaSuccess) return cuda_fail(ctx, e);
    ctx->plan_uploaded = true;
  }
  return AUDIOKV_OK;
}

// Starts the per-kernel timing of one call (event 0), when profiling is on.
void profile_begin(audiokv_ctx* ctx, cudaStream_t stream) {
  Profiler& pf = ctx->prof;
  if (!pf.on) return;
  pf.n = 0;
  cudaEventRecord(pf.ev[0], stream);
  pf.name[0] = "begin";
  pf.n = 1;
}

const ReqDesc* d_reqs(audiokv_ctx* c) { return reinterpret_cast<const ReqDesc*>(c->ws + c->plan.lay.reqs); }
int* d_status(audiokv_ctx* c) { return reinterpret_cast<int*>(c->ws + c->plan.lay.status); }

// head_end >= 0 (one request, tensor-core path only): the heads [head_begin, head_end) alone.
int do_score(audiokv_ctx* ctx, const void* q, const void* k, float* scores, cudaStream_t stream, int head_begin = 0,
             int head_end = -1, bool beside = false) {
  Plan& pl = ctx->plan;
  Launch ln{stream, &ctx->launches, &ctx->prof};
  float2* stats = reinterpret_cast<float2*>(ctx->ws + pl.lay.stats);
  cudaError_t e = cudaErrorNotSupported;
  if (score_umma_takes(pl.sh))
  {
    e = launch_score_umma(pl.sh, pl.reqs.data(), reinterpret_cast<const ScoreUnit*>(ctx->ws + pl.lay.units),
                          reinterpret_cast<const int32_t*>(ctx->ws + pl.lay.ctas), pl.schedules.data(),
                          static_cast<int>(pl.schedules.size()), q, k, scores, stats, pl.score_parts, d_status(ctx), ln,
                          head_begin, head_end, &ctx->score_maps, ctx->plan_id, beside);
  }
  if (head_end >= 0 && e != cudaSuccess) return cuda_fail(ctx, e);  // no head ranges in the FMA kernel
  ctx->score_path = 1;
  if (e == cudaErrorNotSupported) {
    // fp32 inputs (which must not be rounded to TF32), a GQA group above 256 query heads, or strides the copy
    // engine cannot take; audiokv_last_score_path tells the caller which route ran
    ctx->score_path = 2;
    e = launch_score_simt(pl.sh, d_reqs(ctx), q, k, scores, stats, pl.n_slab, kSlabKeys, ln);
  }
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

// Smoothing; with budgets, cu_kept and kept_idx it also selects each head's kept tokens (smoothed may then be null).
// head_end < 0: all heads, in the plan's cost-sorted order; else the heads [head_begin, head_end) in index order.
int do_smooth(audiokv_ctx* ctx, const float* scores, float* smoothed, int32_t* kstar, const int32_t* budgets,
              const int32_t* cu_kept, int32_t* kept_idx, cudaStream_t stream, int head_begin = 0, int head_end = -1) {
  Plan& pl = ctx->plan;
  Launch ln{stream, &ctx->launches, &ctx->prof};
  const bool all = head_end < 0;
  const int count = all ? static_cast<int>(pl.sss_order.size()) : head_end - head_begin;
  cudaError_t e = launch_sss(pl.sh, d_reqs(ctx), reinterpret_cast<const FftPlan*>(ctx->ws + pl.lay.plans),
                             reinterpret_cast<const float2*>(ctx->ws + pl.lay.tables), scores, smoothed, kstar,
                             reinterpret_cast<float2*>(ctx->ws + pl.lay.fft_scratch), pl.scratch_per_block,
                             all ? pl.sss_grid : (count < pl.sss_grid ? count : pl.sss_grid), pl.sss_smem,
                             all ? reinterpret_cast<const int32_t*>(ctx->ws + pl.lay.order) : nullptr, count,
                             head_begin, budgets, cu_kept, kept_idx, d_status(ctx), ln);
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

int do_gather(audiokv_ctx* ctx, const int32_t* cu_kept, const int32_t* kept_idx, const void* k, const void* v,
              void* k_out, void* v_out, cudaStream_t stream, int head_begin = 0, int head_end = -1) {
  Plan& pl = ctx->plan;
  Launch ln{stream, &ctx->launches, &ctx->prof};
  cudaError_t e = launch_gather(pl.sh, d_reqs(ctx), cu_kept, kept_idx, k, v, k_out, v_out, head_begin,
                                head_end < 0 ? pl.sh.total_heads : head_end, ln);
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

int check_budgets(const Plan& pl, const int64_t* total_budget) {
  if (!total_budget) return AUDIOKV_EINVAL;
  const int64_t N = pl.sh.heads_per_req, f = static_cast<int64_t>(pl.sh.window) + pl.sh.base_per_head;
  for (int r = 0; r < pl.sh.n_req; ++r) {
    if (f > pl.reqs[r].L) return AUDIOKV_EINVAL;
    if (total_budget[r] < N * f || total_budget[r] > N * pl.reqs[r].L) return AUDIOKV_EINVAL;
  }
  return AUDIOKV_OK;
}

int do_allocate(audiokv_ctx* ctx, const float* head_scores, const int64_t* total_budget, int32_t* budgets,
                int32_t* cu_kept, cudaStream_t stream) {
  Plan& pl = ctx->plan;
  int rc = check_budgets(pl, total_budget);
  if (rc) return rc;
  Launch ln{stream, &ctx->launches, &ctx->prof};
  cudaError_t e = launch_allocate(pl.sh, d_reqs(ctx), head_scores, total_budget, budgets, cu_kept, d_status(ctx), ln);
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

int do_select_gather(audiokv_ctx* ctx, const float* smoothed, const int32_t* budgets, const int32_t* cu_kept,
                     const void* k, const void* v, void* k_out, void* v_out, int32_t* kept_idx, cudaStream_t stream) {
  Plan& pl = ctx->plan;
  Launch ln{stream, &ctx->launches, &ctx->prof};
  cudaError_t e = launch_select(pl.sh, d_reqs(ctx), smoothed, budgets, cu_kept, kept_idx, pl.max_P, d_status(ctx), ln);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return do_gather(ctx, cu_kept, kept_idx, k, v, k_out, v_out, stream);
}

}  // namespace

extern "C" {

size_t audiokv_params_size(void) { return sizeof(audiokv_params); }

const char* audiokv_strerror(int status) {
  switch (status) {
    case AUDIOKV_OK: return "ok";
    case AUDIOKV_EINVAL: return "invalid argument";
    case AUDIOKV_EALIGN: return "pointer or stride not 16-byte aligned";
    case AUDIOKV_EUNSUPPORTED: return "shape not supported";
    case AUDIOKV_EWORKSPACE: return "workspace too small";
    case AUDIOKV_ECUDA: return "CUDA runtime error";
    case AUDIOKV_ETIMEOUT: return "a kernel gave up a bounded wait";
    case AUDIOKV_EDEVICE: return "a kernel found an index out of range";
    default: return "unknown status";
  }
}

int64_t audiokv_budget_from_ratio(double c, int32_t n_heads_total, int32_t seq_len, int32_t window) {
  if (!(c >= 0.0 && c <= 1.0) || n_heads_total < 1 || seq_len < 1 || window < 0 || window > seq_len) return -1;
  const int64_t hi = static_cast<int64_t>(n_heads_total) * seq_len, lo = static_cast<int64_t>(n_heads_total) * window;
  int64_t b = static_cast<int64_t>(floor(c * static_cast<double>(hi)));
  return b < lo ? lo : (b > hi ? hi : b);
}

int64_t audiokv_scores_len(const audiokv_params* p) {
  int rc = check_params(p);
  if (rc) return rc;
  int64_t n = 0;
  for (int r = 0; r < p->n_req; ++r)
    n += static_cast<int64_t>(p->n_layers) * p->n_kv_heads * (p->seq_len[r] - p->window);
  return n;
}

size_t audiokv_workspace_bytes(const audiokv_params* p) {
  Plan pl;
  if (build_plan(p, &pl)) return 0;
  return pl.lay.end;
}

size_t audiokv_workspace_bytes_host(const audiokv_params* p, int64_t q_elems, int64_t kv_elems,
                                    const int64_t* total_budget) {
  Plan pl;
  if (build_plan(p, &pl) || !total_budget || q_elems < 0 || kv_elems < 0) return 0;
  const size_t es = esize(p->dtype);
  int64_t rows = 0;
  for (int r = 0; r < p->n_req; ++r) rows += total_budget[r];
  size_t off = pl.lay.end;
  off = align_up(off + q_elems * es);
  off = align_up(off + kv_elems * es) ;
  off = align_up(off + kv_elems * es);
  off = align_up(off + sizeof(float) * pl.sh.total_heads);
  off = align_up(off + rows * p->head_dim * es);
  off = align_up(off + rows * p->head_dim * es);
  off = align_up(off + rows * sizeof(int32_t));
  off = align_up(off + sizeof(int32_t) * pl.sh.total_heads);
  off = align_up(off + sizeof(int32_t) * (pl.sh.total_heads + 1));
  return off;
}

int audiokv_create(audiokv_ctx** out, int device, size_t workspace_bytes) {
  if (!out || workspace_bytes == 0) return AUDIOKV_EINVAL;
  *out = nullptr;
  if (cudaSetDevice(device) != cudaSuccess) return AUDIOKV_ECUDA;
  audiokv_ctx* c = new audiokv_ctx();
  c->device = device;
  if (cudaMalloc(&c->ws, workspace_bytes) != cudaSuccess) {
    delete c;
    return AUDIOKV_ECUDA;
  }
  c->ws_bytes = workspace_bytes;
  if (workspace_bytes < 64 || cudaMemset(c->ws, 0, 64) != cudaSuccess) {  // the status word starts clean
    cudaFree(c->ws);
    delete c;
    return workspace_bytes < 64 ? AUDIOKV_EINVAL : AUDIOKV_ECUDA;
  }
  if (cudaEventCreateWithFlags(&c->plan_ready, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->join, cudaEventDisableTiming) != cudaSuccess ||
      cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess) {
    if (c->plan_ready) cudaEventDestroy(c->plan_ready);
    if (c->fork) cudaEventDestroy(c->fork);
    if (c->join) cudaEventDestroy(c->join);
    cudaFree(c->ws);
    delete c;
    return AUDIOKV_ECUDA;
  }
  bool ok = cudaStreamCreateWithFlags(&c->out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&c->copies_out, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < audiokv_ctx::kMaxChunks && ok; ++i)
    ok = cudaEventCreateWithFlags(&c->chunk_in[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&c->chunk_done[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    audiokv_destroy(c);
    return AUDIOKV_ECUDA;
  }
  *out = c;
  return AUDIOKV_OK;
}

int audiokv_destroy(audiokv_ctx* ctx) {
  if (!ctx) return AUDIOKV_EINVAL;
  cudaSetDevice(ctx->device);
  cudaEventDestroy(ctx->plan_ready);
  cudaEventDestroy(ctx->fork);
  cudaEventDestroy(ctx->join);
  cudaStreamDestroy(ctx->side);
  if (ctx->out) cudaStreamDestroy(ctx->out);
  if (ctx->copies_out) cudaEventDestroy(ctx->copies_out);
  for (int i = 0; i < audiokv_ctx::kMaxChunks; ++i) {
    if (ctx->chunk_in[i]) cudaEventDestroy(ctx->chunk_in[i]);
    if (ctx->chunk_done[i]) cudaEventDestroy(ctx->chunk_done[i]);
  }
  for (cudaEvent_t e : ctx->prof.ev)
    if (e) cudaEventDestroy(e);
  cudaFree(ctx->ws);
  delete ctx;
  return AUDIOKV_OK;
}

int audiokv_last_device_status(audiokv_ctx* ctx, audiokv_stream stream) {
  if (!ctx) return AUDIOKV_EINVAL;
  int st = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&st, ctx->ws, sizeof(int), cudaMemcpyDeviceToHost, s);  // first word of the workspace
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess && st != 0) e = cudaMemsetAsync(ctx->ws, 0, sizeof(int), s);  // reported once, then clean again
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return st;
}

const char* audiokv_last_cuda_error(const audiokv_ctx* ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

int64_t audiokv_launch_count(const audiokv_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* audiokv_last_score_path(const audiokv_ctx* ctx) {
  if (!ctx || ctx->score_path == 0) return "none";
  return ctx->score_path == 1 ? "tcgen05" : "fma";
}

int64_t audiokv_set_wait_limit(int64_t cycles) {
  const int64_t before = score_wait_cycles();
  set_score_wait_cycles(cycles);
  return before;
}

int audiokv_profile_enable(audiokv_ctx* ctx, int on) {
  if (!ctx) return AUDIOKV_EINVAL;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return AUDIOKV_ECUDA;
  Profiler& pf = ctx->prof;
  if (on && !pf.ev[0]) {
    for (cudaEvent_t& e : pf.ev)
      if (cudaEventCreate(&e) != cudaSuccess) return AUDIOKV_ECUDA;
  }
  pf.on = on != 0;
  pf.n = 0;
  return AUDIOKV_OK;
}

int audiokv_profile_count(const audiokv_ctx* ctx) { return ctx && ctx->prof.n > 0 ? ctx->prof.n - 1 : 0; }

const char* audiokv_profile_name(const audiokv_ctx* ctx, int i) {
  if (!ctx || i < 0 || i + 1 >= ctx->prof.n) return "";
  return ctx->prof.name[i + 1];
}

float audiokv_profile_ms(audiokv_ctx* ctx, int i) {
  if (!ctx || i < 0 || i + 1 >= ctx->prof.n) return -1.f;
  float ms = -1.f;
  if (cudaEventSynchronize(ctx->prof.ev[i + 1]) != cudaSuccess) return -1.f;
  if (cudaEventElapsedTime(&ms, ctx->prof.ev[i], ctx->prof.ev[i + 1]) != cudaSuccess) return -1.f;
  return ms;
}

int audiokv_score(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k, float* scores,
                  audiokv_stream stream) {
  if (!q_win || !k || !scores) return AUDIOKV_EINVAL;
  if (!aligned16(q_win) || !aligned16(k)) return AUDIOKV_EALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  return do_score(ctx, q_win, k, scores, s);
}

int audiokv_smooth(audiokv_ctx* ctx, const audiokv_params* p, const float* scores, float* smoothed,
                   int32_t* kstar_or_null, audiokv_stream stream) {
  if (!scores || !smoothed) return AUDIOKV_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  return do_smooth(ctx, scores, smoothed, kstar_or_null, nullptr, nullptr, nullptr, s);
}

int audiokv_allocate(audiokv_ctx* ctx, const audiokv_params* p, const float* head_scores,
                     const int64_t* total_budget, int32_t* budgets, int32_t* cu_kept, audiokv_stream stream) {
  if (!head_scores || !total_budget || !budgets || !cu_kept) return AUDIOKV_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  return do_allocate(ctx, head_scores, total_budget, budgets, cu_kept, s);
}

int audiokv_select_gather(audiokv_ctx* ctx, const audiokv_params* p, const float* smoothed, const int32_t* budgets,
                          const int32_t* cu_kept, const void* k, const void* v, void* k_out, void* v_out,
                          int32_t* kept_idx, audiokv_stream stream) {
  if (!smoothed || !budgets || !cu_kept || !k || !v || !k_out || !v_out || !kept_idx) return AUDIOKV_EINVAL;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out)) return AUDIOKV_EALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  return do_select_gather(ctx, smoothed, budgets, cu_kept, k, v, k_out, v_out, kept_idx, s);
}

int audiokv_evict(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k, const void* v,
                  const float* head_scores, const int64_t* total_budget, void* k_out, void* v_out,
                  int32_t* kept_idx, int32_t* budgets, int32_t* cu_kept, audiokv_stream stream) {
  if (!q_win || !k || !v || !head_scores || !total_budget || !k_out || !v_out || !kept_idx || !budgets || !cu_kept)
    return AUDIOKV_EINVAL;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return AUDIOKV_EALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  Plan& pl = ctx->plan;
  float* ws_scores = reinterpret_cast<float*>(ctx->ws + pl.lay.scores);
  int32_t* ws_kstar = reinterpret_cast<int32_t*>(ctx->ws + pl.lay.kstar);
  profile_begin(ctx, s);
  // The budgets depend on nothing the GPU computes, and only the selection needs them. The allocation kernel is
  // launched the ordinary way (everything earlier on the stream is then complete when it starts) and lets its
  // dependents in at once; the first scoring sweep, a programmatic dependent, runs beside it and waits for it at its
  // own end, so that the smoothing and selection, two chained kernels later, find the budgets complete. With per-kernel
  // timing on, every kernel waits for the one before it.
  const bool beside = !ctx->prof.on && score_umma_takes(pl.sh);
  rc = do_allocate(ctx, head_scores, total_budget, budgets, cu_kept, s);
  if (!rc) rc = do_score(ctx, q_win, k, ws_scores, s, 0, -1, beside);
  if (rc) return rc;
  // the pooling variants hand their result to the selection through the score buffer itself
  float* ws_smoothed = pl.sh.smooth_mode >= AUDIOKV_SMOOTH_AVG_POOL ? ws_scores : nullptr;
  if ((rc = do_smooth(ctx, ws_scores, ws_smoothed, ws_kstar, budgets, cu_kept, kept_idx, s))) return rc;
  return do_gather(ctx, cu_kept, kept_idx, k, v, k_out, v_out, s);
}

int audiokv_evict_kstar(audiokv_ctx* ctx, int32_t* kstar, audiokv_stream stream) {
  if (!ctx || !kstar) return AUDIOKV_EINVAL;
  if (!ctx->plan.valid || !ctx->plan_uploaded) return AUDIOKV_EINVAL;  // no pass has run on this context yet
  cudaError_t e = cudaSetDevice(ctx->device);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  e = cudaMemcpyAsync(kstar, ctx->ws + ctx->plan.lay.kstar, sizeof(int32_t) * ctx->plan.sh.total_heads,
                      cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

int audiokv_evict_budgeted(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k, const void* v,
                           const int32_t* budgets, void* k_out, void* v_out, int32_t* kept_idx, int32_t* cu_kept,
                           audiokv_stream stream) {
  if (!q_win || !k || !v || !budgets || !k_out || !v_out || !kept_idx || !cu_kept) return AUDIOKV_EINVAL;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return AUDIOKV_EALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  Plan& pl = ctx->plan;
  float* ws_scores = reinterpret_cast<float*>(ctx->ws + pl.lay.scores);
  int32_t* ws_kstar = reinterpret_cast<int32_t*>(ctx->ws + pl.lay.kstar);
  int32_t* ws_budgets = reinterpret_cast<int32_t*>(ctx->ws + pl.lay.aux);  // the checked copy the selection reads
  profile_begin(ctx, s);
  Launch ln{s, &ctx->launches, &ctx->prof};
  cudaError_t e = launch_budget_prefix(pl.sh, d_reqs(ctx), budgets, ws_budgets, cu_kept, d_status(ctx), ln);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if ((rc = do_score(ctx, q_win, k, ws_scores, s, 0, -1, !ctx->prof.on && score_umma_takes(pl.sh)))) return rc;
  float* ws_smoothed = pl.sh.smooth_mode >= AUDIOKV_SMOOTH_AVG_POOL ? ws_scores : nullptr;
  if ((rc = do_smooth(ctx, ws_scores, ws_smoothed, ws_kstar, ws_budgets, cu_kept, kept_idx, s))) return rc;
  return do_gather(ctx, cu_kept, kept_idx, k, v, k_out, v_out, s);
}

namespace {

// The per-head problem of a re-eviction: every head of the compacted cache becomes a request of one layer and one
// KV head, with its own length, its own place in the packed cache and its own slice of the window queries.
int reevict_problem(ReevictArrays* a, const audiokv_params* p, const int32_t* cu_cache, const int32_t* new_budgets,
                    audiokv_params* dp) {
  if (!a || !p || !cu_cache) return AUDIOKV_EINVAL;
  if (p->n_layers < 1 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->n_q_heads % p->n_kv_heads || p->n_req < 1 ||
      p->head_dim < 1)
    return AUDIOKV_EINVAL;
  const int64_t TH = static_cast<int64_t>(p->n_req) * p->n_layers * p->n_kv_heads;
  if (TH > AUDIOKV_MAX_REQ) return AUDIOKV_EUNSUPPORTED;
  const int G = p->n_q_heads / p->n_kv_heads;
  a->len.resize(TH);
  a->kv_off.resize(TH);
  a->q_off.resize(TH);
  a->budget.resize(TH);
  if (cu_cache[0] != 0) return AUDIOKV_EINVAL;
  int64_t u = 0;
  for (int r = 0; r < p->n_req; ++r) {
    const int64_t q_r = p->q_req_offset ? p->q_req_offset[r] : r * p->q_stride_req;
    for (int l = 0; l < p->n_layers; ++l)
      for (int h = 0; h < p->n_kv_heads; ++h, ++u) {
        const int64_t n = static_cast<int64_t>(cu_cache[u + 1]) - cu_cache[u];
        if (n <= p->window || n > AUDIOKV_MAX_SEQ_LEN) return AUDIOKV_EINVAL;
        a->len[u] = static_cast<int32_t>(n);
        a->kv_off[u] = static_cast<int64_t>(cu_cache[u]) * p->head_dim;
        a->q_off[u] = q_r + l * p->q_stride_layer + static_cast<int64_t>(h) * G * p->q_stride_head;
        if (new_budgets) {
          if (new_budgets[u] < p->window || new_budgets[u] > n) return AUDIOKV_EINVAL;
          a->budget[u] = new_budgets[u];
        }
      }
  }
  *dp = *p;
  dp->n_req = static_cast<int32_t>(TH);
  dp->n_layers = 1;
  dp->n_kv_heads = 1;
  dp->n_q_heads = G;
  dp->seq_len = a->len.data();
  dp->q_stride_req = 0;
  dp->q_stride_layer = 0;
  dp->kv_stride_layer = 0;
  dp->kv_stride_head = 0;
  dp->kv_stride_tok = p->head_dim;
  dp->kv_req_offset = a->kv_off.data();
  dp->q_req_offset = a->q_off.data();
  dp->base_per_head = 0;
  dp->page_size = 0;  // the compacted cache is packed, not paged
  dp->n_pages = 0;
  dp->page_table = nullptr;
  dp->page_table_stride = 0;
  return AUDIOKV_OK;
}

}  // namespace

size_t audiokv_reevict_workspace_bytes(const audiokv_params* p, const int32_t* cu_cache) {
  ReevictArrays tmp;
  audiokv_params dp;
  if (reevict_problem(&tmp, p, cu_cache, nullptr, &dp)) return 0;
  return audiokv_workspace_bytes(&dp);
}

int audiokv_reevict(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k_cache,
                    const void* v_cache, const int32_t* cu_cache, const int32_t* new_budgets, void* k_out, void* v_out,
                    int32_t* kept_idx, int32_t* cu_kept, audiokv_stream stream) {
  if (!ctx || !new_budgets) return AUDIOKV_EINVAL;
  audiokv_params dp;
  int rc = reevict_problem(&ctx->re, p, cu_cache, new_budgets, &dp);
  if (rc) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if ((rc = prepare(ctx, &dp, s))) return rc;
  // One head per request: the allocation hands each its whole total, whatever the weight. The weights and the
  // per-head budgets it writes live in the workspace.
  const size_t TH = ctx->re.len.size();
  float* weights = reinterpret_cast<float*>(ctx->ws + ctx->plan.lay.aux);
  int32_t* budgets = reinterpret_cast<int32_t*>(weights + TH);
  cudaError_t e = cudaMemsetAsync(weights, 0x3f, sizeof(float) * TH, s);  // 0x3f3f3f3f = 0.747
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return audiokv_evict(ctx, &dp, q_win, k_cache, v_cache, weights, ctx->re.budget.data(), k_out, v_out, kept_idx,
                       budgets, cu_kept, s);
}

int audiokv_hit_score(audiokv_ctx* ctx, const float* attn, int32_t n_steps, int32_t n_heads, int64_t row_stride,
                      const int32_t* row_len, const int32_t* span, int32_t top_k, int32_t* hit_counts, float* s_hit,
                      audiokv_stream stream) {
  if (!ctx || !attn || !row_len || !span || !hit_counts || !s_hit) return AUDIOKV_EINVAL;
  if (n_steps < 1 || n_heads < 1 || row_stride < 1 || top_k < 1 || top_k > 1024) return AUDIOKV_EINVAL;
  if (static_cast<int64_t>(n_steps) * n_heads > 0x7fffffffLL || ctx->ws_bytes < 64) return AUDIOKV_EINVAL;
  cudaError_t e = cudaSetDevice(ctx->device);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Launch ln{s, &ctx->launches, &ctx->prof};
  // the status word is the first thing in the workspace, whatever plan the context holds
  e = launch_hit_score(attn, n_steps, n_heads, row_stride, row_len, span, top_k, hit_counts, s_hit,
                       reinterpret_cast<int*>(ctx->ws), ln);
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

int audiokv_selection_spread(audiokv_ctx* ctx, const audiokv_params* p, const int32_t* kept_idx,
                             const int32_t* cu_kept, int32_t n_bins, int32_t* hist, float* stats,
                             audiokv_stream stream) {
  if (!kept_idx || !cu_kept || !hist || !stats) return AUDIOKV_EINVAL;
  if (n_bins < 1 || n_bins > 4096) return AUDIOKV_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  Launch ln{s, &ctx->launches, &ctx->prof};
  cudaError_t e = launch_selection_spread(ctx->plan.sh, d_reqs(ctx), kept_idx, cu_kept, n_bins, hist, stats,
                                          d_status(ctx), ln);
  return e == cudaSuccess ? AUDIOKV_OK : cuda_fail(ctx, e);
}

int audiokv_evict_host(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, int64_t q_elems, const void* k,
                       const void* v, int64_t kv_elems, const float* head_scores, const int64_t* total_budget,
                       void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets, int32_t* cu_kept,
                       audiokv_stream stream) {
  if (!q_win || !k || !v || !head_scores || !total_budget || !k_out || !v_out || !kept_idx || !budgets || !cu_kept)
    return AUDIOKV_EINVAL;
  if (p && p->page_size != 0) return AUDIOKV_EUNSUPPORTED;  // a page table is device data: use audiokv_evict
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(ctx, p, s);
  if (rc) return rc;
  Plan& pl = ctx->plan;
  if (audiokv_workspace_bytes_host(p, q_elems, kv_elems, total_budget) > ctx->ws_bytes) return AUDIOKV_EWORKSPACE;
  const size_t es = esize(p->dtype);
  int64_t rows = 0;
  for (int r = 0; r < p->n_req; ++r) rows += total_budget[r];
  const int TH = pl.sh.total_heads;
  size_t off = pl.lay.end;
  char* dq = ctx->ws + off;   off = align_up(off + q_elems * es);
  char* dk = ctx->ws + off;   off = align_up(off + kv_elems * es);
  char* dv = ctx->ws + off;   off = align_up(off + kv_elems * es);
  char* dS = ctx->ws + off;   off = align_up(off + sizeof(float) * TH);
  char* dko = ctx->ws + off;  off = align_up(off + rows * p->head_dim * es);
  char* dvo = ctx->ws + off;  off = align_up(off + rows * p->head_dim * es);
  char* dki = ctx->ws + off;  off = align_up(off + rows * sizeof(int32_t));
  char* db = ctx->ws + off;   off = align_up(off + sizeof(int32_t) * TH);
  char* dcu = ctx->ws + off;
  cudaError_t e;
#define AKV_CP_ON(st, dst, src, n, kind) \
  if ((e = cudaMemcpyAsync(dst, src, n, kind, st)) != cudaSuccess) return cuda_fail(ctx, e)
#define AKV_CP(dst, src, n, kind) AKV_CP_ON(s, dst, src, n, kind)
  // One request whose K and V are laid out layer by layer, scored on the tensor cores: the pass runs in chunks of
  // layers, so that the copy of the next chunk's K and V (in), this chunk's kernels, and the copy of the previous
  // chunk's kept rows (out) overlap; in and out use the two directions of the link. Everything else: in, pass, out.
  const int NL = pl.sh.n_layers, Hkv = pl.sh.n_kv_heads;
  const bool layered = pl.sh.n_req == 1 && NL > 1 && score_umma_takes(pl.sh) && !ctx->prof.on &&
                       p->kv_stride_layer > 0 && kv_elems == static_cast<int64_t>(NL) * p->kv_stride_layer &&
                       p->kv_stride_layer >= p->kv_stride_tok * pl.reqs[0].L && p->kv_stride_layer >= p->kv_stride_head * Hkv;
  if (layered) {
    const int n_chunks = host_chunks(NL);
    int32_t* d_budgets = reinterpret_cast<int32_t*>(db);
    int32_t* d_cu = reinterpret_cast<int32_t*>(dcu);
    AKV_CP(dq, q_win, q_elems * es, cudaMemcpyHostToDevice);
    AKV_CP(dS, head_scores, sizeof(float) * TH, cudaMemcpyHostToDevice);
    if ((rc = do_allocate(ctx, reinterpret_cast<float*>(dS), total_budget, d_budgets, d_cu, s))) return rc;
    // the chunk boundaries of the output: the prefix sums come back first (a few hundred bytes)
    AKV_CP(budgets, db, sizeof(int32_t) * TH, cudaMemcpyDeviceToHost);
    AKV_CP(cu_kept, dcu, sizeof(int32_t) * (TH + 1), cudaMemcpyDeviceToHost);
    if ((e = cudaEventRecord(ctx->fork, s)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(ctx, e);
    // the copy streams start behind everything the caller's stream holds so far (the workspace may be in use)
    if ((e = cudaStreamWaitEvent(ctx->side, ctx->fork, 0)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaStreamWaitEvent(ctx->out, ctx->fork, 0)) != cudaSuccess) return cuda_fail(ctx, e);
    float* ws_scores = reinterpret_cast<float*>(ctx->ws + pl.lay.scores);
    int32_t* ws_kstar = reinterpret_cast<int32_t*>(ctx->ws + pl.lay.kstar);
    float* ws_smoothed = pl.sh.smooth_mode >= AUDIOKV_SMOOTH_AVG_POOL ? ws_scores : nullptr;
    const size_t layer_bytes = static_cast<size_t>(p->kv_stride_layer) * es, row_bytes = static_cast<size_t>(p->head_dim) * es;
    // V is only ever read by the gather, and only its kept rows: when the caller's V is pinned memory the device can
    // address, the gather fetches those rows straight from it and the rest of V never crosses the link.
    const void* v_src = dv;
    {
      cudaPointerAttributes at{};
      if (cudaPointerGetAttributes(&at, v) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer &&
          aligned16(at.devicePointer))
        v_src = at.devicePointer;
      else
        cudaGetLastError();  // pageable memory is reported as an error by older drivers: not one of this call's
    }
    for (int c = 0; c < n_chunks; ++c) {
      const int l0 = host_chunk_layer(NL, c), l1 = host_chunk_layer(NL, c + 1);
      const size_t off = l0 * layer_bytes, len = (l1 - l0) * layer_bytes;
      AKV_CP_ON(ctx->side, dk + off, static_cast<const char*>(k) + off, len, cudaMemcpyHostToDevice);
      if (v_src == dv) AKV_CP_ON(ctx->side, dv + off, static_cast<const char*>(v) + off, len, cudaMemcpyHostToDevice);
      if ((e = cudaEventRecord(ctx->chunk_in[c], ctx->side)) != cudaSuccess) return cuda_fail(ctx, e);
      if ((e = cudaStreamWaitEvent(s, ctx->chunk_in[c], 0)) != cudaSuccess) return cuda_fail(ctx, e);
      const int u0 = l0 * Hkv, u1 = l1 * Hkv;
      if ((rc = do_score(ctx, dq, dk, ws_scores, s, u0, u1))) return rc;
      if ((rc = do_smooth(ctx, ws_scores, ws_smoothed, ws_kstar, d_budgets, d_cu, reinterpret_cast<int32_t*>(dki), s, u0, u1)))
        return rc;
      if ((rc = do_gather(ctx, d_cu, reinterpret_cast<int32_t*>(dki), dk, v_src, dko, dvo, s, u0, u1))) return rc;
      if ((e = cudaEventRecord(ctx->chunk_done[c], s)) != cudaSuccess) return cuda_fail(ctx, e);
      if ((e = cudaStreamWaitEvent(ctx->out, ctx->chunk_done[c], 0)) != cudaSuccess) return cuda_fail(ctx, e);
      const size_t r0 = static_cast<size_t>(cu_kept[u0]), r1 = static_cast<size_t>(cu_kept[u1]);  // host copy, read above
      AKV_CP_ON(ctx->out, static_cast<char*>(k_out) + r0 * row_bytes, dko + r0 * row_bytes, (r1 - r0) * row_bytes,
                cudaMemcpyDeviceToHost);
      AKV_CP_ON(ctx->out, static_cast<char*>(v_out) + r0 * row_bytes, dvo + r0 * row_bytes, (r1 - r0) * row_bytes,
                cudaMemcpyDeviceToHost);
      AKV_CP_ON(ctx->out, reinterpret_cast<char*>(kept_idx) + r0 * sizeof(int32_t), dki + r0 * sizeof(int32_t),
                (r1 - r0) * sizeof(int32_t), cudaMemcpyDeviceToHost);
    }
    // the caller's stream ends behind the last copy out, then the host waits for it
    if ((e = cudaEventRecord(ctx->copies_out, ctx->out)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaStreamWaitEvent(s, ctx->copies_out, 0)) != cudaSuccess) return cuda_fail(ctx, e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(ctx, e);
    return AUDIOKV_OK;
  }
  AKV_CP(dq, q_win, q_elems * es, cudaMemcpyHostToDevice);
  AKV_CP(dk, k, kv_elems * es, cudaMemcpyHostToDevice);
  AKV_CP(dv, v, kv_elems * es, cudaMemcpyHostToDevice);
  AKV_CP(dS, head_scores, sizeof(float) * TH, cudaMemcpyHostToDevice);
  rc = audiokv_evict(ctx, p, dq, dk, dv, reinterpret_cast<float*>(dS), total_budget, dko, dvo,
                     reinterpret_cast<int32_t*>(dki), reinterpret_cast<int32_t*>(db), reinterpret_cast<int32_t*>(dcu), s);
  if (rc) return rc;
  AKV_CP(k_out, dko, rows * p->head_dim * es, cudaMemcpyDeviceToHost);
  AKV_CP(v_out, dvo, rows * p->head_dim * es, cudaMemcpyDeviceToHost);
  AKV_CP(kept_idx, dki, rows * sizeof(int32_t), cudaMemcpyDeviceToHost);
  AKV_CP(budgets, db, sizeof(int32_t) * TH, cudaMemcpyDeviceToHost);
  AKV_CP(cu_kept, dcu, sizeof(int32_t) * (TH + 1), cudaMemcpyDeviceToHost);
#undef AKV_CP
#undef AKV_CP_ON
  if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(ctx, e);
  return AUDIOKV_OK;
}

}  // extern "C"
