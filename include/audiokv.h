/* audiokv.h -- C boundary of the B200 (sm_100a) AudioKV eviction pass.
 *
 * The pass runs once after prefill. For every request, layer and KV head it
 *   1. scores each prefix token by the attention the last W queries give it
 *      (Section 3.3: the per-head importance sequence over a decoding window),
 *   2. smooths that sequence in the frequency domain (Section 3.3: Spectral Score
 *      Smoothing, the RFFT / energy cut-off / mask / IRFFT / residual-mix equations),
 *   3. turns per-head audio-criticality scores into integer budgets (Section 3.1,
 *      b = w + r + B_score * S / sum S; Section 3.2's floor rule is the case w = r = 0),
 *   4. keeps the top-scoring tokens of each head plus the window and copies their
 *      K and V rows into a compacted cache (the paper's Top-K selection and eviction).
 *
 * Conventions
 *   - Every data pointer is DEVICE memory owned by the caller unless marked "host".
 *     The library allocates only inside audiokv_create and frees only in audiokv_destroy.
 *   - Every compute call is asynchronous on the given CUDA stream, never synchronises
 *     the device and never throws. It returns AUDIOKV_OK or a negative status. Problems
 *     seen by a kernel (a bounded wait that ran out) are written to a status word
 *     that audiokv_last_device_status reads.
 *   - Q, K and V share one element type (`dtype`); the last dimension (head_dim) is
 *     contiguous; bases and strides of K/V/Q rows must be 16-byte aligned.
 *   - L_r is the number of cached tokens of request r (prompt incl. the window),
 *     W the window, P_r = L_r - W the number of eviction candidates (prefix tokens).
 *   - Heads are numbered flat: u = (r * n_layers + l) * n_kv_heads + h.
 *   - Score buffers are fp32, packed: head u of request r starts at
 *       score_offset(r) + (l * n_kv_heads + h) * P_r,
 *     score_offset(r) = sum_{r' < r} n_layers * n_kv_heads * P_{r'};
 *     audiokv_scores_len() gives the total length.
 *   - Compacted outputs are packed in flat head order: head u owns rows
 *     [cu_kept[u], cu_kept[u+1]) of k_out / v_out ([rows][head_dim]) and of kept_idx;
 *     inside a head the kept prefix tokens come in ascending token order, then the
 *     W window tokens.
 */
#ifndef AUDIOKV_H_
#define AUDIOKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { AUDIOKV_F32 = 0, AUDIOKV_BF16 = 1 };

/* Step 2 as the paper defines it, and the variants used for ablation-style runs. */
enum {
  AUDIOKV_SMOOTH_SSS = 0,            /* Spectral Score Smoothing: energy cut-off rho (Section 3.3)              */
  AUDIOKV_SMOOTH_FIXED_FRACTION = 1, /* same filter, cut-off at k* = floor(smooth_kappa * (n/2)): the other     */
                                     /* reading of the cut-off range in the sensitivity study (Section 4.6)     */
  AUDIOKV_SMOOTH_ENERGY_NO_MEAN = 2, /* energy cut-off with bin 0 left out of the energy (bin 0 always passes)  */
  AUDIOKV_SMOOTH_AVG_POOL = 3,       /* local average pooling over pool_kernel tokens, zero padding: the local  */
  AUDIOKV_SMOOTH_MAX_POOL = 4        /* pooling of the SnapKV lineage that SSS replaces (Sections 3.3, 4.3)     */
};

enum {
  AUDIOKV_OK = 0,
  AUDIOKV_EINVAL = -1,       /* an argument is out of range or inconsistent            */
  AUDIOKV_EALIGN = -2,       /* a pointer or stride breaks the 16-byte rule            */
  AUDIOKV_EUNSUPPORTED = -3, /* shape outside what the kernels are built for           */
  AUDIOKV_EWORKSPACE = -4,   /* the context's workspace is too small for these params  */
  AUDIOKV_ECUDA = -5,        /* a CUDA runtime call failed (see audiokv_last_cuda_error)*/
  AUDIOKV_ETIMEOUT = -6,     /* a kernel gave up a bounded wait                        */
  AUDIOKV_EDEVICE = -7       /* a kernel found an index out of range                   */
};

typedef struct audiokv_ctx audiokv_ctx; /* opaque: device workspace, tables, status word */
typedef void* audiokv_stream;           /* a cudaStream_t                                */

/* Problem description; plain data in HOST memory, read during the call only. */
typedef struct {
  int32_t dtype;                 /* AUDIOKV_F32 | AUDIOKV_BF16                                   */
  int32_t n_layers;              /* layers evicted in this call (>= 1)                           */
  int32_t n_q_heads;             /* query heads per layer; a multiple of n_kv_heads              */
  int32_t n_kv_heads;
  int32_t head_dim;              /* 64, 128 or 256                                               */
  int32_t n_req;                 /* requests in the (ragged) batch, 1..AUDIOKV_MAX_REQ           */
  const int32_t* seq_len;        /* host [n_req]: L_r, each > window                             */
  int32_t window;                /* W >= 1: the last W tokens are the observation window         */
  /* element (not byte) offsets: Q(r,l,i,a,t) = r*q_stride_req + l*q_stride_layer + i*q_stride_tok + a*q_stride_head + t */
  int64_t q_stride_req, q_stride_layer, q_stride_tok, q_stride_head;
  /* K/V(r,l,h,j,t) = kv_req_offset[r] + l*kv_stride_layer + h*kv_stride_head + j*kv_stride_tok + t */
  int64_t kv_stride_layer, kv_stride_tok, kv_stride_head;
  const int64_t* kv_req_offset;  /* host [n_req], or NULL for all-zero                           */
  float softmax_scale;           /* <= 0 selects 1/sqrt(head_dim)                                */
  float rho;                     /* SSS energy cut-off ratio, in (0, 1]                          */
  float alpha;                   /* SSS mixing coefficient, in [0, 1]                            */
  int32_t transition_bins;       /* T >= 0: cosine band of T bins after the cut-off; 0 = binary mask */
  int32_t base_per_head;         /* r >= 0: uniform base allocation per head, in tokens          */
  /* Smoothing variant (all zero = the paper's method). See audiokv_smooth.                            */
  int32_t smooth_mode;           /* AUDIOKV_SMOOTH_*                                             */
  float smooth_kappa;            /* AUDIOKV_SMOOTH_FIXED_FRACTION: cut-off fraction in [0, 1]    */
  int32_t pool_kernel;           /* AUDIOKV_SMOOTH_*_POOL: odd window, 1 .. 1023 tokens          */
  const int64_t* q_req_offset;   /* host [n_req], or NULL: element offset of request r's window queries,
                                    replacing r*q_stride_req (which is then ignored)              */
  /* Paged K/V (page_size = 0: off). K and V are then pools of n_pages pages of page_size tokens, and
   * K/V(r,l,h,j,t) = l*kv_stride_layer + h*kv_stride_head + (page_table[r][j / page_size]*page_size
   * + j % page_size)*kv_stride_tok + t; kv_req_offset is ignored. Tokens of a page beyond L_r may hold
   * anything. A page id outside [0, n_pages) is not followed: AUDIOKV_EDEVICE in the status word.   */
  int32_t page_size;             /* 0, 16, 32, 64 or 128 tokens                                  */
  int32_t n_pages;               /* pages in the pool                                            */
  const int32_t* page_table;     /* DEVICE int32 [n_req][page_table_stride], read when the kernels run;
                                    request r uses its first ceil(L_r / page_size) entries        */
  int64_t page_table_stride;     /* >= ceil(max L / page_size)                                   */
} audiokv_params;

#define AUDIOKV_MAX_REQ 8192
#define AUDIOKV_MAX_SEQ_LEN 131072

/* ---- host-side helpers (no GPU work) ------------------------------------------------ */

/* sizeof(audiokv_params) as the library was built: a binding in another language compares
 * it with the size of its own copy of the struct before the first call. */
size_t audiokv_params_size(void);

/* Text for a status code. Never NULL. */
const char* audiokv_strerror(int status);

/* Total kept rows of one request at retention ratio c (the paper's "KV-cache retention
 * ratio"): floor(c * n_heads_total * L), clamped to [n_heads_total * window, n_heads_total * L].
 * n_heads_total = n_layers * n_kv_heads. Compute it once and hand the same integer to
 * every consumer. Returns -1 for arguments out of range. */
int64_t audiokv_budget_from_ratio(double c, int32_t n_heads_total, int32_t seq_len, int32_t window);

/* Number of fp32 elements of a packed score buffer for these params (sum_r N * P_r), or a
 * negative status. */
int64_t audiokv_scores_len(const audiokv_params* p);

/* Bytes of workspace audiokv_create must be given so that every call below works for
 * these params (0 on invalid params). Grows with sum_r L_r; a few MB per 100k tokens. */
size_t audiokv_workspace_bytes(const audiokv_params* p);

/* ---- context ------------------------------------------------------------------------- */

/* Creates a context on `device` with a workspace of `workspace_bytes` (cudaMalloc; the only
 * allocation the library makes). *ctx is set on success. */
int audiokv_create(audiokv_ctx** ctx, int device, size_t workspace_bytes);

/* Threads and streams: a context holds one plan, one workspace and the tensor maps of its last
 * call, so calls on ONE context must not run concurrently, neither from two host threads nor on
 * two streams whose work may overlap on the GPU (their kernels would share the score buffers).
 * Use one context per stream; contexts are independent of one another.
 *
 * Stream capture: every device-buffer entry point may be recorded into a CUDA graph, once the
 * context has seen its params in a call OUTSIDE capture (the first call with a new shape copies
 * the plan up from pageable memory and waits for it; inside a capture it returns AUDIOKV_ECUDA
 * and says so in audiokv_last_cuda_error). Every kernel of audiokv_evict goes to the caller's stream
 * (some as programmatic dependents of the one before). The host-buffer call waits on the host and
 * cannot be captured. */

/* Frees the workspace. The caller makes sure no call on this context is still running. */
int audiokv_destroy(audiokv_ctx* ctx);

/* The status word the kernels write (0, AUDIOKV_ETIMEOUT, AUDIOKV_EDEVICE or, from
 * audiokv_evict_budgeted, AUDIOKV_EINVAL). Synchronises with the work of earlier calls by a
 * blocking copy on `stream`; a non-zero status is reported once and the word is cleared. */
int audiokv_last_device_status(audiokv_ctx* ctx, audiokv_stream stream);

/* Text of the last CUDA error a call on this context met (empty string if none). */
const char* audiokv_last_cuda_error(const audiokv_ctx* ctx);

/* Kernels launched by calls on this context since it was created (for accounting). */
int64_t audiokv_launch_count(const audiokv_ctx* ctx);

/* Which kernels the last scoring on this context ran on (audiokv_score, or step 1 inside audiokv_evict and
 * its variants): "tcgen05" = the tensor-core kernels (bf16 inputs), "fma" = the fp32 FMA kernels (fp32
 * inputs, which are never rounded to TF32; a GQA group of more than 256 query heads; row strides the copy
 * engine cannot express), "none" before the first scoring. Never NULL. */
const char* audiokv_last_score_path(const audiokv_ctx* ctx);

/* Limit of the waits inside the tensor-core scoring kernels (the paper has no counterpart: this is the
 * library's guard against a wait that never ends). Every wait of a warp on a barrier of its CTA gives up
 * after `cycles` SM clock cycles (default 2e9, about a second): the CTA then stops, lets its copies and
 * tensor-core operations in flight finish, releases its tensor memory, and the kernel writes
 * AUDIOKV_ETIMEOUT to the status word; the call's outputs are then undefined and the context stays usable.
 * Process-wide, read at each launch; cycles <= 0 restores the default. Returns the previous limit. Meant for
 * deployments that want a shorter guard and for the test that makes a wait run out. */
int64_t audiokv_set_wait_limit(int64_t cycles);

/* Per-kernel timing of audiokv_evict, for benchmarks. While enabled, every audiokv_evict call
 * on this context records a CUDA event on its stream after each kernel it launches (creating
 * the events on the first enable). After the call, kernel i of the call (0 <= i <
 * audiokv_profile_count) has the name audiokv_profile_name(ctx, i) and took
 * audiokv_profile_ms(ctx, i) milliseconds from the end of the kernel before it (blocks until
 * that kernel has finished; -1 on error). Off by default. */
int audiokv_profile_enable(audiokv_ctx* ctx, int on);
int audiokv_profile_count(const audiokv_ctx* ctx);
const char* audiokv_profile_name(const audiokv_ctx* ctx, int i);
float audiokv_profile_ms(audiokv_ctx* ctx, int i);

/* ---- the four steps ------------------------------------------------------------------- */

/* Step 1 -- importance scores (Section 3.3, importance sequence over the decoding window).
 * For window row i (token P+i), query head a of KV head h's group and key j <= P+i:
 *   z = softmax_scale * <Q[i,a,:], K[j,h,:]>, p = softmax over the visible j; then
 *   scores_h[j] = sum over the W rows and the group's query heads of p, for j < P.
 * q_win: the window's queries (layout by q_stride_*). k: the key cache (kv_stride_*).
 * scores: packed fp32 output (see top). bf16 inputs use tensor cores with fp32
 * accumulation; f32 inputs use fp32 FMA (no TF32). */
int audiokv_score(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k, float* scores,
                  audiokv_stream stream);

/* Step 2 -- Spectral Score Smoothing (Section 3.3). Per head, on x = scores (length n = P):
 *   F = RFFT(x); E(k) = sum_{i<=k} |F_i|^2; k* = min{k : E(k) >= rho * E(n/2)};
 *   w_i = 1 (i <= k*), (1 + cos(pi (i-k*)/(T+1)))/2 (k* < i <= k*+T), 0 beyond;
 *   x~ = IRFFT(F .* w, n); smoothed = (1 - alpha) x + alpha x~.
 * Any n >= 1 (mixed radix for smooth lengths, chirp-z otherwise). `smoothed` may equal
 * `scores`. kstar_or_null: optional int32 [total heads] receiving k* (0 for the pooling modes).
 * Variants (smooth_mode): FIXED_FRACTION and ENERGY_NO_MEAN change only how k* is chosen;
 * AVG_POOL / MAX_POOL replace x~ by the pooled sequence y_j = mean (zero padding counted) or
 * max of x over |i - j| <= pool_kernel / 2; the residual mix with alpha is the same. */
int audiokv_smooth(audiokv_ctx* ctx, const audiokv_params* p, const float* scores, float* smoothed,
                   int32_t* kstar_or_null, audiokv_stream stream);

/* Step 3 -- head-wise budgets (Section 3.1 allocation rule; Section 3.2's rule when
 * window and base are taken out). Per request, over its N = n_layers * n_kv_heads heads:
 * every head gets window + base_per_head rows; the rest of total_budget[r] is shared in
 * proportion to head_scores (integer arithmetic on round(S * 2^24): floors, then the
 * left-over rows by largest remainder, lower head index first); no head exceeds L_r
 * (excess is re-shared). The budgets of a request add up to total_budget[r] exactly.
 * head_scores: device fp32 [n_req][n_layers][n_kv_heads], each in [0, 128].
 * total_budget: HOST int64 [n_req], N*(W+base) <= B_r <= N*L_r (else AUDIOKV_EINVAL).
 * budgets: device int32 [total heads] (window included).
 * cu_kept: device int32 [total heads + 1], exclusive prefix sum of budgets. */
int audiokv_allocate(audiokv_ctx* ctx, const audiokv_params* p, const float* head_scores,
                     const int64_t* total_budget, int32_t* budgets, int32_t* cu_kept, audiokv_stream stream);

/* Step 4 -- Top-K selection and eviction. Per head u: the budgets[u] - W prefix tokens
 * with the largest smoothed score (ties: lower token index), in ascending token order,
 * then the window tokens P..L-1; their indices go to kept_idx and their K and V rows,
 * copied bit for bit, to k_out and v_out, all at rows [cu_kept[u], cu_kept[u+1]).
 * k_out / v_out must not overlap k / v. NaN scores give an unspecified selection. */
int audiokv_select_gather(audiokv_ctx* ctx, const audiokv_params* p, const float* smoothed, const int32_t* budgets,
                          const int32_t* cu_kept, const void* k, const void* v, void* k_out, void* v_out,
                          int32_t* kept_idx, audiokv_stream stream);

/* The whole pass in one call: allocate, score, smooth, select, gather, with the
 * intermediate score buffers in the context's workspace. Arguments as above; budgets and
 * cu_kept are outputs. k_out, v_out and kept_idx need sum_r total_budget[r] rows. */
int audiokv_evict(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k, const void* v,
                  const float* head_scores, const int64_t* total_budget, void* k_out, void* v_out,
                  int32_t* kept_idx, int32_t* budgets, int32_t* cu_kept, audiokv_stream stream);

/* The cut-offs k* of step 2 as the last audiokv_evict / audiokv_evict_budgeted / audiokv_reevict call on
 * this context found them (Section 3.3, the smallest k with E(k) >= rho E(n/2); 0 for the pooling
 * variants): a copy of the context's own record, ordered on `stream` behind that call.
 * kstar: device int32 [total heads]. AUDIOKV_EINVAL before the first pass on the context. */
int audiokv_evict_kstar(audiokv_ctx* ctx, int32_t* kstar, audiokv_stream stream);

/* Same pass with every buffer in HOST memory (pageable or pinned): copies the inputs to
 * the device (into the workspace, which must have been sized with
 * audiokv_workspace_bytes_host), runs the pass, copies kept_idx, budgets, cu_kept,
 * k_out and v_out back and waits for the stream. q/k/v extents are given in elements.
 * One bf16 request whose K and V are laid out layer by layer (kv_elems = n_layers *
 * kv_stride_layer) is processed in chunks of layers on three streams of the context, so
 * that copies in, kernels and copies out overlap; when v is pinned memory the device can
 * address, the kept V rows are read from it in place and the rest of V is never copied.
 * Results do not depend on the route taken. Paged K/V (page_size != 0) is not accepted
 * here (AUDIOKV_EUNSUPPORTED): the page table is device data. */
int audiokv_evict_host(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, int64_t q_elems, const void* k,
                       const void* v, int64_t kv_elems, const float* head_scores, const int64_t* total_budget,
                       void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets, int32_t* cu_kept,
                       audiokv_stream stream);
size_t audiokv_workspace_bytes_host(const audiokv_params* p, int64_t q_elems, int64_t kv_elems,
                                    const int64_t* total_budget);

/* The pass with budgets chosen by the caller: steps 1, 2 and 4 of audiokv_evict, step 3 left
 * out. For a run that shards the heads over several GPUs (the allocation of Section 3.1
 * normalises over ALL layers and heads of a request, so it is computed once for the whole
 * stack with audiokv_allocate and each GPU evicts its layers with its slice of the result),
 * and for budget rules other than the paper's.
 * budgets: device int32 [total heads], W <= budgets[u] <= L_r; a value outside is clamped
 * into that range and reported as AUDIOKV_EINVAL in the status word. cu_kept is an output
 * (prefix sums of the budgets); k_out, v_out, kept_idx need sum_u budgets[u] rows. */
int audiokv_evict_budgeted(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k, const void* v,
                           const int32_t* budgets, void* k_out, void* v_out, int32_t* kept_idx, int32_t* cu_kept,
                           audiokv_stream stream);

/* Decode-time re-eviction of an already compacted cache (Section 3.3: the importance
 * sequence may also come from a sliding window of decoding steps; Fig. 3, decoding phase).
 * After an eviction every head has its own length, so the cache is ragged per head: head
 * u = (r*n_layers + l)*n_kv_heads + h holds rows [cu_cache[u], cu_cache[u+1]) of k_cache
 * and v_cache (device, [rows][head_dim], row stride head_dim) in token order, the tokens
 * decoded since the last eviction appended at the end; the last `window` rows are the
 * tokens whose queries q_win holds (layout and strides as in audiokv_score). The call runs
 * steps 1, 2 and 4 on every head with its own length n_u: scores of the first n_u - W rows,
 * smoothing, the new_budgets[u] - W best of them plus the window, gathered.
 *   p: dtype, n_layers, n_q_heads, n_kv_heads, head_dim, n_req, window, the q strides
 *      (and q_req_offset), softmax_scale and the smoothing fields are read; seq_len, the kv
 *      strides, kv_req_offset and base_per_head are ignored.
 *   cu_cache: HOST int32 [total heads + 1], cu_cache[0] = 0, every n_u in (W, AUDIOKV_MAX_SEQ_LEN].
 *   new_budgets: HOST int32 [total heads], W <= new_budgets[u] <= n_u: rows head u keeps.
 *   k_out / v_out: device, sum_u new_budgets[u] rows; kept_idx: device int32, as many entries,
 *      positions inside the head's own cache rows, ascending; cu_kept: device int32
 *      [total heads + 1], the prefix sums of new_budgets.
 * total heads <= AUDIOKV_MAX_REQ (else AUDIOKV_EUNSUPPORTED). The context's workspace must hold
 * audiokv_reevict_workspace_bytes(p, cu_cache) bytes (0 on invalid arguments). */
size_t audiokv_reevict_workspace_bytes(const audiokv_params* p, const int32_t* cu_cache);
int audiokv_reevict(audiokv_ctx* ctx, const audiokv_params* p, const void* q_win, const void* k_cache,
                    const void* v_cache, const int32_t* cu_cache, const int32_t* new_budgets, void* k_out, void* v_out,
                    int32_t* kept_idx, int32_t* cu_kept, audiokv_stream stream);

/* Selection spread (Section 1, the figure on the distribution of Top-K selections before
 * and after smoothing): where along the prefix the kept tokens of a request's heads fall.
 * Token j of request r's prefix belongs to stretch floor(j * n_bins / P_r); hist[r][b]
 * counts, over the request's n_layers * n_kv_heads heads, the kept prefix tokens in
 * stretch b (window tokens are not counted). stats[r] = {balance, peak}:
 *   balance = -sum_b p_b ln p_b / ln n_bins, p_b = hist[r][b] / sum_b hist[r][b]
 *             (1 = flat, 0 = one stretch; 0 when n_bins = 1),
 *   peak    = max_b hist[r][b] * n_bins / sum_b hist[r][b];  both 0 when nothing is kept.
 * kept_idx, cu_kept: device, as audiokv_evict / audiokv_select_gather wrote them.
 * n_bins: 1..4096. hist: device int32 [n_req][n_bins]; stats: device fp32 [n_req][2]. */
int audiokv_selection_spread(audiokv_ctx* ctx, const audiokv_params* p, const int32_t* kept_idx,
                             const int32_t* cu_kept, int32_t n_bins, int32_t* hist, float* stats,
                             audiokv_stream stream);

/* Offline head score (Section 3.2, "Collecting Attention Hits to Audio Spans" and "Head Importance
 * Estimation"): the table S that audiokv_allocate consumes. For decode step t and head a, with
 * S = TopK(attention row, top_k) (ties: lower token index) and the inclusive audio-token span
 * [span[2t], span[2t+1]] of the word generated at step t:
 *   c = |S intersect span|,  r = c / top_k,  s_hit[a] = mean over the steps of r.
 * attn: device fp32 [n_steps][n_heads][row_stride], row t holds row_len[t] <= row_stride tokens (a row
 * shorter than top_k contributes all of them). row_len: device int32 [n_steps]. span: device int32
 * [n_steps][2]. top_k in 1..1024 (the paper uses 24). hit_counts: device int32 [n_heads], receives the
 * integer totals sum_t c. s_hit: device fp32 [n_heads]. The paper records the rows with hooks on a real
 * model and takes the spans from a word aligner; neither is part of this library. */
int audiokv_hit_score(audiokv_ctx* ctx, const float* attn, int32_t n_steps, int32_t n_heads, int64_t row_stride,
                      const int32_t* row_len, const int32_t* span, int32_t top_k, int32_t* hit_counts, float* s_hit,
                      audiokv_stream stream);

/* Step 1 for callers that cannot allocate device memory (the paper has no counterpart: this
 * is a deployment variant of audiokv_score, same arguments and same result).
 * Who needs it: code running under a memory pool or arena whose owner forbids cudaMalloc
 * once serving has started, plug-ins that receive a stream and buffers but no allocator, and
 * callers that must avoid the device-wide synchronisation an allocation may cause. It takes
 * no context: its scratch (the per-slab softmax statistics and the request table) is a fixed
 * 8 MiB array inside the library image, which every GPU that loads the library holds until
 * the process exits. It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - Limits: n_req <= 64 (more is AUDIOKV_EINVAL), and
 *     n_req * n_layers * n_kv_heads * ceil(max L / 512) * W * G * 8 bytes must fit in
 *     8 MiB - 4 KiB (e.g. 28 layers x 4 KV heads at L = 8192, W = 32, G = 7 needs 3.1 MiB);
 *     larger problems return AUDIOKV_EWORKSPACE. fp32 FMA arithmetic for both element types.
 *   - The first call on a device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on one GPU share the array: two calls whose kernels may overlap on the GPU
 *     (different streams without an ordering between them) race on it. Calls ordered on one
 *     stream are safe; nothing needs clearing between calls, since the first kernel writes every
 *     scratch entry the second one reads.
 * device: CUDA device ordinal (made current). Other arguments as audiokv_score. */
int audiokv_score_noalloc(int device, const audiokv_params* p, const void* q_win, const void* k, float* scores,
                          audiokv_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* AUDIOKV_H_ */
