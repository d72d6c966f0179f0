// Importance scores for bf16 inputs on the tcgen05 tensor cores (sm_100a).
//
// The score of key j is the sum, over the W window rows and the G query heads of a KV
// head, of softmax probabilities. A column sum mixes rows with different normalisers,
// so the keys are swept twice:
//   sweep 1  D[row][key]  = Q K^T  (query rows on the TMEM lanes): every thread owns one
//            row (two, when W * G exceeds 128) and keeps a reference and a sum of exp2 over
//            the keys of its tiles; one pair per (head, part, group, row) goes to the
//            statistics buffer.
//   sweep 2  D[key][row]  = K Q^T  (keys on the TMEM lanes): every thread owns one key
//            and adds exp2(z - max - log2 sum) over its set's rows; the two sets' sums of a key meet in the score
//            buffer (atomic adds into a buffer that sweep 1 cleared).
// Both sweeps are one persistent kernel with three roles:
//   warps 0-15  two epilogue groups of two sets of four warps (one warp per TMEM lane quarter and set). The groups
//               take the tiles of the CTA in turn (group g the tiles with parity g), each through accumulator
//               buffers of its own, so that they depend on nothing but their MMA thread: no barrier joins them,
//               nothing is exchanged through shared memory, and while one group waits, loads or stores, the other
//               keeps the special-function unit busy. The two sets of a group split the columns of every part;
//   warp 16     TMA producer: the Q tile of a head once, K tiles of 128 keys through a ring;
//   warps 17-18 MMA issuers, one thread per epilogue group: tcgen05.mma, bf16 x bf16 -> fp32 in TMEM. With one issuer
//               for both groups the tiles were issued in order, and a group that had handed its buffers back waited
//               for the MMAs of the other group's tile to be let in first.
// A tile is processed in one or two parts (sweep 1: blocks of 128 query rows; sweep 2: halves of
// the query rows), each with an accumulator buffer of 128 TMEM columns that goes back to the MMA
// thread as soon as its last chunk is in registers: the MMAs of the group's next tile run under
// the arithmetic of this one.
// The work of a launch is dealt out tile by tile: CTA c takes the tiles [c T / grid, (c + 1) T / grid)
// of the launch's tile sequence, as a few runs of consecutive tiles of one head (host-built table).
// Q and K tiles are K-major with the 128-byte swizzle, so the same shared-memory tile is
// the A operand of one sweep and the B operand of the other.
// Every wait on an mbarrier is bounded: when one runs out the CTA stops, the kernel
// writes AUDIOKV_ETIMEOUT to the status word and returns with its TMEM released.
#include <cuda.h>
#include <stddef.h>

#include <atomic>

#include "common.cuh"

namespace akv {
namespace {

constexpr int kTileKeys = 128;    // keys per K tile (UMMA M in sweep 2, N in sweep 1)
// Epilogue warps: two groups of kSets sets of four warps (one warp per TMEM lane quarter); the sets of a group split
// the columns of every part. Both sweeps run two sets (four epilogue warps per scheduler, 96 registers per thread).
// Sweep 1: 92 us against 104 with one set (its maxima leave the special-function unit idle often enough for a second
// pair of warps per scheduler to pay). Sweep 2 ran one set with 168 registers and 64-column steps for a long time
// (85 us; two sets on the same steps 90: no registers left to schedule with); two sets on 32-column steps, with the
// same share of the exponentials on the FMA pipe, take 80 us. After the epilogue warps come the producer warp and
// the two MMA warps.
constexpr int epi_sets(int sweep) { return 2; }
constexpr int epi_warps(int sweep) { return 8 * epi_sets(sweep); }
constexpr int n_threads(int sweep) { return (epi_warps(sweep) + 3) * 32; }
constexpr int kStatSets = 2 * epi_sets(1);  // statistics entries sweep 1 writes per part: [group][set]
constexpr uint32_t kTmemCols = 512;  // four accumulator buffers of 128 columns: [group][buffer]
constexpr int kMaxStages = 8;
constexpr long long kWaitCycles = 2000000000LL;  // about one second: default limit of every wait on an mbarrier
constexpr long long kDrainCycles = 200000000LL;  // limit of the waits of the stop path (copies and MMAs still in flight)
constexpr int kSmemLimit = 232448;               // 227 KB

// Tensor maps travel as kernel arguments, CAP requests' worth per launch. Two sizes: 8 for the usual small batch (the
// arguments are copied at every launch, and 31 KB of them cost each sweep about 1.5 us), 120 for long batches such
// as one request per head (32 KB of arguments at most).
constexpr int kMapChunkSmall = 8, kMapChunkLarge = 120;

template <int CAP>
struct TmapPack {
  CUtensorMap q[CAP];  // 4-D per request: (d, query head, window row, layer)
  CUtensorMap k[CAP];  // 4-D per request: (d, token, KV head, layer)
};

struct UmmaArgs {
  Shape sh;
  const ScoreUnit* units;    // this sweep's runs, in processing order
  const int32_t* cta_begin;  // [grid + 1]: CTA c takes the runs cta_begin[c] .. cta_begin[c + 1] - 1
  float2* stats;
  float* scores;
  int* status;
  int max_parts;  // statistics slots per head: [head][part][group][row]
  int q_rows;     // rows of the Q tile in shared memory: 128 or 256
  int r_pad;      // query rows of a Q tile rounded up to 16
  int n_stages;   // K ring depth
  int r0;         // first request of this launch: request r uses maps q[r - r0], k[r - r0]
  int w_chunk;    // window rows of a run's Q tile (the whole window, or a share of it when W * G exceeds the tile)
  int accumulate; // sweep 2 adds into `scores` (cleared by sweep 1): two warp sets per key, or several chunks of window rows
  int beside;     // sweep 1 runs beside the kernel launched before it (see launch_score_umma) and waits for it at its end
  long long wait_cycles;  // limit of a wait on an mbarrier, in SM clock cycles
};

struct Small {
  alignas(16) float negc[2][2][256];  // sweep 2: -(max + log2 sum) per row: [group][head parity][row]
  alignas(8) uint64_t k_full[kMaxStages];
  uint64_t k_empty[kMaxStages];
  uint64_t q_full, q_empty;
  uint64_t acc_full[2][2], acc_empty[2][2];  // [group][buffer]
  uint64_t grp_bar[2];  // the 128 threads of a group (sweep 2: the rows' normalisers of a new head are in place)
  uint64_t drain[2];    // stop path only: the MMAs of either issuer still in flight
  uint32_t tmem_base;
  int abort;
};
static_assert(sizeof(TmapPack<kMapChunkLarge>) + sizeof(UmmaArgs) <= 32764, "kernel arguments are limited to 32764 bytes");
static_assert(offsetof(Small, negc) % 16 == 0 && offsetof(Small, k_full) % 8 == 0, "alignment of the small shared area");

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// May suspend the thread, for a time of the hardware's choosing, until the phase completes. (An explicit suspend-time
// hint was measured and made the sweeps a fifth slower: the default wake-up is the quicker one.)
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// The same question without suspending the thread.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false when the CTA is stopping (this or another wait ran out). try_wait may suspend the
// thread for a time of the hardware's choosing before it answers, which is what a long wait wants; with a limit
// shorter than such a suspension the barrier is polled instead, so that the limit is what ends the wait.
constexpr long long kPollBelow = 1000000LL;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, long long limit) {
  const bool poll = limit < kPollBelow;
  if (poll ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!(poll ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity))) {
    if (poll || (++spins & 15u) == 0) {  // a try_wait that comes back empty-handed has slept a while already
      if (*abort) return false;
      if (clock64() - t0 > limit) {
        *abort = 1;
        return false;
      }
    }
  }
  return true;
}
// Wait of the stop path: the CTA is already stopping, so the flag is not consulted; bounded all the same.
__device__ __forceinline__ void mbar_wait_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > kDrainCycles) return;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// The same copy with an L2 eviction hint: `policy` comes from l2_evict_first().
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// Shared-memory matrix descriptor of a K-major bf16 tile with the 128-byte swizzle: rows of
// 128 bytes, groups of 8 rows 1024 bytes apart. `saddr` may point 32 * k bytes into the
// first row to select the k-th slice of 16 elements along K.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);  // start address
  d |= static_cast<uint64_t>(1) << 16;                          // leading-dimension offset (unused here)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                  // stride between 8-row groups
  d |= static_cast<uint64_t>(1) << 46;                          // descriptor version of sm_100
  d |= static_cast<uint64_t>(2) << 61;                          // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, tile M x N.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 (16) consecutive fp32 columns of this thread's TMEM lane. The load is asynchronous: the
// registers hold the data only after tmem_wait on the same array (the first wait after a batch
// of loads waits for all of them), so a thread issues every load of a tile up front.
#define AKV_R8(r, o) "=r"(r[o]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define AKV_RW8(r, o) "+r"(r[o]), "+r"(r[o + 1]), "+r"(r[o + 2]), "+r"(r[o + 3]), "+r"(r[o + 4]), "+r"(r[o + 5]), "+r"(r[o + 6]), "+r"(r[o + 7])
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : AKV_R8(r, 0), AKV_R8(r, 8), AKV_R8(r, 16), AKV_R8(r, 24)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
      : AKV_R8(r, 0), AKV_R8(r, 8)
      : "r"(taddr)
      : "memory");
}
// The same for 16 columns, into the low half of a 32-register buffer.
__device__ __forceinline__ void tmem_ld16_issue_lo(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
      : AKV_R8(r, 0), AKV_R8(r, 8)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_lo(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" : AKV_RW8(r, 0), AKV_RW8(r, 8)::"memory");
}
__device__ __forceinline__ void tmem_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" : AKV_RW8(r, 0), AKV_RW8(r, 8), AKV_RW8(r, 16), AKV_RW8(r, 24)::"memory");
}
__device__ __forceinline__ void tmem_wait(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" : AKV_RW8(r, 0), AKV_RW8(r, 8)::"memory");
}
#undef AKV_R8
#undef AKV_RW8

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Two fp32 values in one 64-bit register: the scale-and-shift before an exponential and the add after
// it are issued once per pair (fma.rn.f32x2 / add.rn.f32x2), which leaves issue slots to the
// special-function unit that bounds both sweeps.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ f32x2 pack2(uint32_t a, uint32_t b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// exp2 of both halves
__device__ __forceinline__ f32x2 ex2_2(f32x2 x) {
  float a, b;
  unpack2(x, a, b);
  return pack2(ex2(a), ex2(b));
}
__device__ __forceinline__ float hsum(f32x2 a, f32x2 b, f32x2 c, f32x2 d) {
  float x, y;
  unpack2(add2(add2(a, b), add2(c, d)), x, y);
  return x + y;
}

// exp2 on the FMA pipe, for a share of the exponentials: the special-function unit delivers 16 exp2 per clock and
// SM and bounds both sweeps, while the FMA pipe has room. With t = round(x) + 1.5 * 2^23 (the integer lands in the low
// mantissa bits), n = t - 1.5 * 2^23 and f = x - n in [-1/2, 1/2]: 2^x = 2^n p(f), p the cubic that minimises the
// maximum relative error of 2^f on that interval (7.5e-5; rms 5e-5, well inside the 1e-3 the scores are held to),
// and 2^n is an integer add into the exponent field. x must lie in [-125, 2^22).
constexpr float kMagic = 12582912.f;  // 1.5 * 2^23
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// x and t = round(x) + kMagic, both halves
__device__ __forceinline__ f32x2 ex2_poly(f32x2 x, f32x2 t) {
  const f32x2 f = sub2(x, sub2(t, pack2(kMagic, kMagic)));
  f32x2 p = fma2(f, pack2(5.5171664930e-02f, 5.5171664930e-02f), pack2(2.4261112188e-01f, 2.4261112188e-01f));
  p = fma2(p, f, pack2(6.9326098622e-01f, 6.9326098622e-01f));
  p = fma2(p, f, pack2(9.9992807358e-01f, 9.9992807358e-01f));
  uint32_t tl, th, pl, ph;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(tl), "=r"(th) : "l"(t));
  asm("mov.b64 {%0, %1}, %2;" : "=r"(pl), "=r"(ph) : "l"(p));
  return pack2(pl + (tl << 23), ph + (th << 23));
}
// Of every eight pairs of exponentials, this many go to the FMA pipe. In the kernel as it stands (four epilogue warps
// per scheduler in both sweeps): sweep 2 takes 87.2 us with none, 80.9 with one, 79.9 with two, 83.8 with three;
// sweep 1, once its per-step maxima were gone, 86.6 with none, 84.8 with one, 85.5 with two, 88.4 with three.
#ifndef AKV_POLY_S1
#define AKV_POLY_S1 1
#endif
#ifndef AKV_POLY_S2
#define AKV_POLY_S2 2
#endif
constexpr int kPolyS1 = AKV_POLY_S1, kPolyS2 = AKV_POLY_S2;

// Sweep 1 works on 64 accumulator columns of a row at a time (two register buffers of 32).
__device__ __forceinline__ float max32(const uint32_t (&r)[32]) {
  float c0 = max3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
  float c1 = max3(__uint_as_float(r[3]), __uint_as_float(r[4]), __uint_as_float(r[5]));
  float c2 = max3(__uint_as_float(r[6]), __uint_as_float(r[7]), __uint_as_float(r[8]));
  float c3 = max3(__uint_as_float(r[9]), __uint_as_float(r[10]), __uint_as_float(r[11]));
#pragma unroll
  for (int i = 12; i + 7 < 32; i += 8) {
    c0 = max3(c0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
    c1 = max3(c1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
    c2 = max3(c2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
    c3 = max3(c3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
  }
  c0 = max3(c0, __uint_as_float(r[28]), __uint_as_float(r[29]));
  c1 = max3(c1, __uint_as_float(r[30]), __uint_as_float(r[31]));
  return fmaxf(max3(c0, c1, c2), c3);
}
// Adds exp2(r * sl - m) of 32 logits into four pairs of partial sums; m is a whole number of octaves.
__device__ __forceinline__ void exp_sum32(const uint32_t (&r)[32], float sl, float inv_sl, float m, f32x2& a0, f32x2& a1,
                                          f32x2& a2, f32x2& a3) {
  const float nb = -m;
  const float r_min = (m - 120.f) * inv_sl;  // logits below this add less than 2^-120 each: held there for the polynomial
  const f32x2 sl2 = pack2(sl, sl), nb2 = pack2(nb, nb), nbm2 = pack2(nb + kMagic, nb + kMagic);
#pragma unroll
  for (int i = 0; i < 32; i += 16) {
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      const uint32_t x0 = r[i + 2 * p], x1 = r[i + 2 * p + 1];
      f32x2 e;
      if (p < kPolyS1) {
        const f32x2 v = pack2(fmaxf(__uint_as_float(x0), r_min), fmaxf(__uint_as_float(x1), r_min));
        e = ex2_poly(fma2(v, sl2, nb2), fma2(v, sl2, nbm2));  // nb is an integer: nb + kMagic is exact
      } else {
        e = ex2_2(fma2(pack2(x0, x1), sl2, nb2));
      }
      if ((p & 3) == 0) a0 = add2(a0, e);
      else if ((p & 3) == 1) a1 = add2(a1, e);
      else if ((p & 3) == 2) a2 = add2(a2, e);
      else a3 = add2(a3, e);
    }
  }
}
// The next whole octave at or above x: adding 1.5 * 2^23 rounded upwards leaves ceil(x) in the low mantissa bits
// (FMA-pipe operations; ceilf would queue behind the exponentials in the special-function unit).
__device__ __forceinline__ float ceil_octave(float x) { return __fadd_ru(x, kMagic) - kMagic; }

// Sweep 1: 64 logits of this thread's row (columns col0 .. col0 + 63 of the tile, in two buffers). Updates the row's
// reference m_ref (a whole number of octaves, so that changing it rescales the sum exactly) and its sum Z of exp2
// relative to that reference. The exponentials are taken against the reference the row had BEFORE these columns:
// a reference tens of octaves away from the maximum loses nothing in fp32, so only the first columns of a run
// look for their maximum first, and only a sum of 2^60 or more (a jump of the maximum by about that much, or an
// overflow) has the exponentials taken once more. Afterwards the reference is raised by what the SUM of the columns
// says (it bounds their maximum from above), which needs no maximum over the columns: measured, the 22 three-input
// maxima per step kept the ALU pipe from taking a share of the exponentials (with them, a polynomial share made
// the sweep slower; without them, one pair in eight on the FMA pipe brings 87.6 -> 84.8 us).
__device__ __forceinline__ void stats_step(uint32_t (&ra)[32], uint32_t (&rb)[32], bool masked, int col0, int last_col,
                                           float sl, float inv_sl, float& m_ref, float& Z) {
  if (masked) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      if (col0 + i > last_col) ra[i] = 0xff800000u;  // -inf
      if (col0 + 32 + i > last_col) rb[i] = 0xff800000u;
    }
  }
  if (m_ref == -INFINITY) {
    const float cm = fmaxf(max32(ra), max32(rb));
    if (cm == -INFINITY) return;  // fully masked: adds nothing
    m_ref = ceil_octave(cm * sl);
  }
  f32x2 a0 = pack2(0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;
  exp_sum32(ra, sl, inv_sl, m_ref, a0, a1, a2, a3);
  exp_sum32(rb, sl, inv_sl, m_ref, a0, a1, a2, a3);
  const float s = hsum(a0, a1, a2, a3);  // these columns' sum relative to m_ref: at least their largest term
  if (!(s < 0x1p60f)) {
    // a jump of the maximum by tens of octaves (or an overflow): take the exponentials again, against the maximum
    const float cm = fmaxf(max32(ra), max32(rb));
    const float m_new = ceil_octave(cm * sl);
    a0 = a1 = a2 = a3 = pack2(0.f, 0.f);
    exp_sum32(ra, sl, inv_sl, m_new, a0, a1, a2, a3);
    exp_sum32(rb, sl, inv_sl, m_new, a0, a1, a2, a3);
    Z = fmaf(Z, ex2(m_ref - m_new), hsum(a0, a1, a2, a3));
    m_ref = m_new;
  } else {
    // Keep the reference above what was seen, so that later columns stay in range: when the sum reaches 1 the
    // reference goes up by the sum's binary exponent + 1 (a whole number of octaves: the rescaling is exact and is
    // built from bits, no special function). The sum bounds the maximum from above, so no maximum is needed.
    const int e = s >= 1.f ? (__float_as_int(s) >> 23) - 126 : 0;            // 0 <= e <= 60
    Z = (Z + s) * __int_as_float((127 - e) << 23);                            // * 2^-e
    m_ref += __int_as_float(0x4b000000 | e) - 8388608.f;                      // + e
  }
}
// Sweep 2: N logits of this thread's key against N query rows; nc = their -(max + log2 sum), 16-byte aligned.
// Adds exp2(z * sl + nc[row]) into four pairs of partial sums. The arguments are at most 0 (up to rounding).
template <int N>
__device__ __forceinline__ void colsum_part(const uint32_t (&r)[32], const float* __restrict__ nc, f32x2 sl2, f32x2& a0,
                                            f32x2& a1, f32x2& a2, f32x2& a3) {
  const ulonglong2* nc2 = reinterpret_cast<const ulonglong2*>(nc);
  const f32x2 magic2 = pack2(kMagic, kMagic);
#pragma unroll
  for (int j = 0; j < N; j += 8) {
    const ulonglong2 v = nc2[j >> 2], w = nc2[(j >> 2) + 1];
    const int n_poly = (j & 8) ? kPolyS2 / 2 : (kPolyS2 + 1) / 2;  // of every 4 pairs, alternately: 1 and 1 make 2 of 8
    f32x2 x[4] = {fma2(pack2(r[j], r[j + 1]), sl2, v.x), fma2(pack2(r[j + 2], r[j + 3]), sl2, v.y),
                  fma2(pack2(r[j + 4], r[j + 5]), sl2, w.x), fma2(pack2(r[j + 6], r[j + 7]), sl2, w.y)};
    f32x2 e[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      if (p < n_poly) {
        float lo, hi;
        unpack2(x[p], lo, hi);
        const f32x2 c = pack2(fmaxf(lo, -120.f), fmaxf(hi, -120.f));  // padding rows carry -inf
        e[p] = ex2_poly(c, add2(c, magic2));
      } else {
        e[p] = ex2_2(x[p]);
      }
    }
    a0 = add2(a0, e[0]);
    a1 = add2(a1, e[1]);
    a2 = add2(a2, e[2]);
    a3 = add2(a3, e[3]);
  }
}

// Sweep 2, set SET of two: the chunks 2 SET and 2 SET + 1 of a part of COLS accumulator columns (a multiple of 16, at
// most 128) for this thread's key, one 32-column buffer at a time; the shape is known at compile time, so the tile
// loop has no branch on chunk counts or on a half-filled last buffer. The part's buffer is handed back to the MMA
// thread once this set's last chunk is in registers (at once when the set has no chunk in the part).
template <int COLS, int SET>
__device__ __forceinline__ void colsum_cols_set(uint32_t taddr, const float* __restrict__ ncp, f32x2 sl2, uint32_t ebar, int lane,
                                                uint32_t (&ra)[32], f32x2& a0, f32x2& a1, f32x2& a2, f32x2& a3) {
  constexpr int n_ch = (COLS + 31) / 32;
  constexpr bool tail = (COLS & 16) != 0;
  constexpr int c_lo = 2 * SET, c_hi = c_lo + 2 < n_ch ? c_lo + 2 : n_ch;  // chunks [c_lo, c_hi)
  if (c_lo >= n_ch) {
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(ebar);
    return;
  }
#pragma unroll
  for (int c = c_lo; c < c_hi; ++c) {
    const bool half = tail && c == n_ch - 1;
    if (half) tmem_ld16_issue_lo(taddr + c * 32, ra);
    else tmem_ld32_issue(taddr + c * 32, ra);
    if (half) tmem_wait_lo(ra);
    else tmem_wait(ra);
    if (c == c_hi - 1) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(ebar);
    }
    if (half) colsum_part<16>(ra, ncp + c * 32, sl2, a0, a1, a2, a3);
    else colsum_part<32>(ra, ncp + c * 32, sl2, a0, a1, a2, a3);
  }
}

template <int SWEEP, int D, int CAP>
__global__ void __launch_bounds__(n_threads(SWEEP), 1)
score_umma_kernel(const __grid_constant__ TmapPack<CAP> tm, const UmmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int KB = D / 64;                 // 64-element (128-byte) blocks along the head dimension
  constexpr int kKBlk = kTileKeys * 128;     // bytes of one such block of a K tile
  constexpr int kKStage = KB * kKBlk;
  const int q_blk = a.q_rows * 128;
  uint8_t* q_s = smem;
  uint8_t* k_s = q_s + KB * q_blk;
  Small* sm = reinterpret_cast<Small*>(k_s + a.n_stages * kKStage);
  volatile int* abort = &sm->abort;

  const Shape& sh = a.sh;
  const int G = sh.group, R = a.w_chunk * G;  // query rows of a run's Q tile; Rt: of the head (statistics layout)
  const int Rt = sh.window * G;
  constexpr int kSets = epi_sets(SWEEP), kEpiWarps = epi_warps(SWEEP), kThreads = n_threads(SWEEP);
  constexpr int kProducerWarp = kEpiWarps, kMmaWarp = kEpiWarps + 1;  // and kEpiWarps + 2: an MMA thread per group
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = a.n_stages;
  const long long wl = a.wait_cycles;
  // Parts of a tile, each with an accumulator buffer of its own.
  //   sweep 1: blocks of 128 query rows (M = 128 rows, N = 128 keys);
  //   sweep 2: the query rows in one piece (up to 128) or in two halves of whole 16s (M = 128 keys, N = the rows).
  const int n_parts = SWEEP == 1 ? (R > 128 ? 2 : 1) : (a.r_pad > 128 ? 2 : 1);
  const int cols0 = SWEEP == 1 ? kTileKeys : (n_parts == 2 ? ((a.r_pad >> 4) + 1) / 2 * 16 : a.r_pad);
  const int cols1 = SWEEP == 1 ? kTileKeys : a.r_pad - cols0;

  // ---- set-up ----
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(smem_u32(&sm->k_full[s]), 1);
      mbar_init(smem_u32(&sm->k_empty[s]), 1);
    }
    mbar_init(smem_u32(&sm->q_full), 1);
    mbar_init(smem_u32(&sm->q_empty), 2);  // both MMA threads are done with the Q tile
    for (int g = 0; g < 2; ++g) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(smem_u32(&sm->acc_full[g][b]), 1);
        mbar_init(smem_u32(&sm->acc_empty[g][b]), 4 * kSets);  // the warps of the group
      }
      mbar_init(smem_u32(&sm->grp_bar[g]), 128 * kSets);
    }
    mbar_init(smem_u32(&sm->drain[0]), 1);
    mbar_init(smem_u32(&sm->drain[1]), 1);
    sm->abort = 0;
    fence_barrier_init();
  }
  {  // rows of the Q tile that no copy ever writes must read as zero
    uint4* qz = reinterpret_cast<uint4*>(q_s);
    const int n16 = KB * q_blk / 16;
    for (int i = threadIdx.x; i < n16; i += kThreads) qz[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
  }
  if (warp == kProducerWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // Everything above is local to the CTA. Sweep 1 now waits for the kernels before it (they may have written K
  // and Q) and only then lets sweep 2 be brought in. A CTA of sweep 2 therefore starts on inputs that are
  // final: its copies and MMAs begin as soon as a CTA of sweep 1 has left the SM, and only its epilogue waits
  // (below) for sweep 1 to finish, since only the statistics come from there.
  // When the kernel before sweep 1 is the library's own budget kernel, launched the ordinary way (so that everything
  // earlier on the stream is complete) and needing nothing sweep 1 touches, sweep 1 runs beside it and waits for it
  // only at its end: the kernels after it then find the budgets complete through the chain of waits.
  if (SWEEP == 1 && !a.beside) chain_wait();
  chain_release();
  const uint32_t tmem_base = sm->tmem_base;

  const int unit_begin = __ldg(a.cta_begin + blockIdx.x), unit_end = __ldg(a.cta_begin + blockIdx.x + 1);

  if (warp == kProducerWarp) {
    // ---- TMA producer ----
    // Lane 0 runs the ring. With a paged pool the 128 / page_size pages of a tile are fetched by as many lanes,
    // one page each (a copy costs its issuing thread about a hundred cycles, and a tile of 16-token pages is 8 to 32
    // copies): those lanes walk the same schedule, lane 0 alone waits and arms the barriers, and its result reaches
    // the others through the shuffle that also orders their copies after the arming.
    const int n_sub = a.sh.page_size ? kTileKeys >> a.sh.page_shift : 1;
    const uint32_t lanes = (1u << n_sub) - 1u;
    if (lane < n_sub) {
      // K tiles are marked evict-first in L2 in both sweeps: a pass streams far more K than L2 holds, and what the
      // next kernels need (scores, tables, statistics, their code) should not be pushed out by the stream. Lines
      // under no pressure stay, so a K that fits in L2 is still found there by sweep 2.
      const uint64_t evict_first = l2_evict_first();
      int it = 0, heads = 0, prev_u = -1, s = 0;  // s, ph: slot of the K ring and its phase
      uint32_t ph = 0;
      bool ok = true;
      ScoreUnit Unext = a.units[unit_begin < unit_end ? unit_begin : 0];
      for (int n = unit_begin; n < unit_end && ok; ++n) {
        const ScoreUnit U = Unext;
        if (n + 1 < unit_end) Unext = a.units[n + 1];  // the next descriptor arrives under this run's work
        for (int t = 0; t < U.n_tiles; ++t, ++it) {
          const uint32_t bar = smem_u32(&sm->k_full[s]);
          int page_y = 0;
          if (a.sh.page_size) {
            // this lane's page of the tile; past the request's last token, or with an id outside the pool (which is
            // reported), the copy starts outside the map and delivers zeros
            const int tok = U.kt0 + t * kTileKeys + lane * a.sh.page_size;
            page_y = a.sh.n_pages << a.sh.page_shift;
            if (tok < U.P + a.sh.window) {
              const int pg = __ldg(a.sh.page_table + U.r * a.sh.page_table_stride + (tok >> a.sh.page_shift));
              if (pg >= 0 && pg < a.sh.n_pages) page_y = pg << a.sh.page_shift;
              else atomicExch(a.status, AUDIOKV_EDEVICE);
            }
          }
          bool mine = true;
          if (lane == 0) {
            if (t == 0 && U.qid != prev_u) {
              if (heads > 0) mine = mbar_wait(smem_u32(&sm->q_empty), (heads - 1) & 1, abort, wl);  // MMAs on the old Q are done
              if (mine) {
                // the box is w_chunk window rows; rows of a last, shorter chunk beyond the window arrive as zeros
                const uint32_t qbar = smem_u32(&sm->q_full);
                mbar_expect_tx(qbar, static_cast<uint32_t>(R) * D * 2);
                for (int kb = 0; kb < KB; ++kb)
                  tma_load_4d(smem_u32(q_s + kb * q_blk), &tm.q[U.r - a.r0], qbar, kb * 64, U.h * G, U.w0, U.l);
                prev_u = U.qid;
                ++heads;
              }
            }
            if (mine) mine = mbar_wait(smem_u32(&sm->k_empty[s]), ph ^ 1, abort, wl);
            if (mine) mbar_expect_tx(bar, kKStage);
          }
          ok = __shfl_sync(lanes, mine, 0);
          if (!ok) break;
          if (a.sh.page_size == 0) {
            for (int kb = 0; kb < KB; ++kb) {
              tma_load_4d_hint(smem_u32(k_s + s * kKStage + kb * kKBlk), &tm.k[U.r - a.r0], bar, kb * 64,
                               U.kt0 + t * kTileKeys, U.h, U.l, evict_first);
            }
          } else {
            // k[0] maps the whole pool as (d, page * page_size + token in page, KV head, layer) with a box of one
            // page: at least 16 rows of 128 bytes, whole swizzle groups, so the tile comes out as in the contiguous case
            for (int kb = 0; kb < KB; ++kb) {
              const uint32_t dst = smem_u32(k_s + s * kKStage + kb * kKBlk + lane * a.sh.page_size * 128);
              tma_load_4d_hint(dst, &tm.k[0], bar, kb * 64, page_y, U.h, U.l, evict_first);
            }
          }
          if (++s == S) {
            s = 0;
            ph ^= 1;
          }
        }
      }
      if (lane == 0 && *abort) {  // let the copies still in flight land before the CTA goes away
        for (int j = it > S ? it - S : 0; j < it; ++j) mbar_wait_drain(smem_u32(&sm->k_full[j % S]), (j / S) & 1);
        if (heads > 0) mbar_wait_drain(smem_u32(&sm->q_full), (heads - 1) & 1);
      }
    }
  } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
    if (lane == 0) {
      // ---- MMA issuer of group g ----
      // Tile `it` of the CTA belongs to group it & 1 and sits in stage it % S of the K ring. Its parts go to the
      // group's buffers in turn: part number qc of the group uses buffer qc & 1, in phase (qc >> 1) & 1 of the
      // buffer's barriers.
      const int g = warp - kMmaWarp;
      int it = 0, heads = 0, prev_u = -1, qc = 0;
      bool ok = true;
      ScoreUnit Unext = a.units[unit_begin < unit_end ? unit_begin : 0];
      for (int n = unit_begin; n < unit_end && ok; ++n) {
        const ScoreUnit U = Unext;
        if (n + 1 < unit_end) Unext = a.units[n + 1];  // the next descriptor arrives under this run's work
        if (U.qid != prev_u) {
          if (prev_u != -1) umma_commit(smem_u32(&sm->q_empty));  // this thread's MMAs on the old Q tile are done
          ok = mbar_wait(smem_u32(&sm->q_full), heads & 1, abort, wl);
          if (!ok) break;
          tc_fence_after();
          prev_u = U.qid;
          ++heads;
        }
        for (int t = 0; t < U.n_tiles && ok; ++t, ++it) {
          if ((it & 1) != g) continue;  // the other thread's tile
          const int s = it % S;
          ok = mbar_wait(smem_u32(&sm->k_full[s]), (it / S) & 1, abort, wl);
          if (!ok) break;
          const uint32_t k_addr = smem_u32(k_s + s * kKStage);
          const uint32_t q_addr = smem_u32(q_s);
          for (int p = 0; p < n_parts; ++p) {
            const int b = qc & 1;
            ok = mbar_wait(smem_u32(&sm->acc_empty[g][b]), ((qc >> 1) & 1) ^ 1, abort, wl);
            if (!ok) break;
            ++qc;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (2 * g + b) * 128;
            // byte offset of the part inside the Q tile (a multiple of 1024: whole 8-row groups)
            const uint32_t q_off = SWEEP == 1 ? p * (128 * 128) : (p == 0 ? 0 : cols0 * 128);
            const uint32_t idesc = SWEEP == 1 ? umma_idesc(128, kTileKeys) : umma_idesc(kTileKeys, p == 0 ? cols0 : cols1);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
              for (int ks = 0; ks < 4; ++ks) {
                const uint64_t dq = umma_desc(q_addr + kb * q_blk + q_off + ks * 32);
                const uint64_t dk = umma_desc(k_addr + kb * kKBlk + ks * 32);
                if (SWEEP == 1) umma_bf16(d_tmem, dq, dk, idesc, (kb | ks) != 0);
                else umma_bf16(d_tmem, dk, dq, idesc, (kb | ks) != 0);
              }
            }
            umma_commit(smem_u32(&sm->acc_full[g][b]));
          }
          if (ok) umma_commit(smem_u32(&sm->k_empty[s]));
        }
      }
      if (*abort) {  // TMEM must not be released under MMAs that are still running
        umma_commit(smem_u32(&sm->drain[g]));
        mbar_wait_drain(smem_u32(&sm->drain[g]), 0);
      }
    }
  } else {
    // ---- epilogue: two groups of kSets sets of four warps; warp w reads TMEM lanes 32 (w % 4) .. +31 ----
    const int g = warp / (4 * kSets), set = (warp >> 2) % kSets, quarter = warp & 3;
    const int gl = quarter * 32 + lane;  // TMEM lane
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + 2 * g * 128;
    const float sl = sh.scale_log2e, inv_sl = 1.0f / sl;
    int it = 0, prev_u = -1, heads = 0, qc = 0;
    uint32_t grp_phase = 0;
    bool ok = true;
    uint32_t ra[32], rb[32];
    if (SWEEP == 2) chain_wait();  // the statistics of sweep 1 are complete and visible
    ScoreUnit Unext = a.units[unit_begin < unit_end ? unit_begin : 0];
    for (int n = unit_begin; n < unit_end && ok; ++n) {
      const ScoreUnit U = Unext;
      if (n + 1 < unit_end) Unext = a.units[n + 1];
      const int live_rows = U.wn * G;  // query rows of this run (the Q tile may hold more: padding, a short last chunk)
      if (SWEEP == 2 && U.qid != prev_u) {
        // Merge the parts' statistics of this head: negc[row] = -(max + log2 sum); padding rows get -inf. Each group
        // keeps a copy of its own, in two versions by head parity: a warp of the group that is still on the head before
        // reads the other version, and none can be two heads behind the barrier below.
        float* dst = sm->negc[g][heads & 1];
        for (int rr = set * 128 + gl; rr < 256; rr += 128 * kSets) {
          float c = -INFINITY;
          if (rr < live_rows) {
            const float2* hs = a.stats + static_cast<int64_t>(U.u) * a.max_parts * kStatSets * Rt + U.w0 * G + rr;
            float M = -INFINITY, Zt = 0.f;
            const int n_ent = U.head_parts * kStatSets;
            for (int s0 = 0; s0 < n_ent; s0 += 8) {
              float2 sv[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                sv[i] = s0 + i < n_ent ? __ldcg(hs + static_cast<int64_t>(s0 + i) * Rt)  // written by the kernel before
                                       : make_float2(-INFINITY, 0.f);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                if (sv[i].y > 0.f) {
                  const float m_new = fmaxf(M, sv[i].x);
                  Zt = Zt * exp2f(M - m_new) + sv[i].y * exp2f(sv[i].x - m_new);  // first: 0 * exp2(-inf) = 0
                  M = m_new;
                }
              }
            }
            c = -(M + log2f(Zt));
          }
          dst[rr] = c;
        }
        ++heads;
        mbar_arrive(smem_u32(&sm->grp_bar[g]));
        ok = mbar_wait(smem_u32(&sm->grp_bar[g]), grp_phase, abort, wl);
        grp_phase ^= 1;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      prev_u = U.qid;
      if (SWEEP == 1 && a.accumulate && U.w0 == 0) {
        // Sweep 2 adds a key's column sums into the score buffer from several places (its two warp sets; the chunks
        // of a window scored in chunks), so the run of the first chunk clears the entries of its keys (sweep 2's
        // epilogue starts after this kernel has ended)
        const int k_end = U.kt0 + U.n_tiles * kTileKeys < U.P ? U.kt0 + U.n_tiles * kTileKeys : U.P;
        for (int key = U.kt0 + static_cast<int>(threadIdx.x); key < k_end; key += kEpiWarps * 32)
          a.scores[U.score_base + key] = 0.f;
      }
      // sweep 1: this thread's rows gl and 128 + gl: reference, in whole octaves, and sum of exp2 relative to it
      float m_ref[2] = {-INFINITY, -INFINITY}, Z[2] = {0.f, 0.f};
      const float* nc = SWEEP == 2 ? sm->negc[g][(heads - 1) & 1] : nullptr;
      for (int t = 0; t < U.n_tiles; ++t, ++it) {
        if ((it & 1) != g) continue;  // the other group's tile
        const int kt = U.kt0 + t * kTileKeys;
        const f32x2 sl2 = pack2(sl, sl);
        f32x2 a0 = pack2(0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;  // sweep 2: this key's sums over the rows
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          if (p >= n_parts || !ok) continue;
          const int b = qc & 1;
          ok = mbar_wait(smem_u32(&sm->acc_full[g][b]), (qc >> 1) & 1, abort, wl);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) continue;
          ++qc;
          tc_fence_after();
          const uint32_t taddr = lane_addr + b * 128;
          const uint32_t ebar = smem_u32(&sm->acc_empty[g][b]);
          // Steps of 64 accumulator columns (two register buffers of 32; the last one may hold 16 in sweep 2): the loads of
          // a step land within tens of cycles, so nothing is prefetched, and the arithmetic of a step is one long block
          // of independent work for the scheduler. The accumulator buffer goes back to the MMA thread as soon as its
          // last step is in registers.
          const int cols = p == 0 ? cols0 : cols1;
          const int n_ch = (cols + 31) >> 5;
          const bool tail = (cols & 16) != 0;
          const int row = p * 128 + gl;                       // sweep 1: this thread's query row in the part
          const bool live = row < live_rows;
          const bool masked = kt + kTileKeys - 1 > U.P;       // sweep 1: the tile reaches into the window: causal mask
          const int last_col = U.P + U.w0 + row / G - kt;     // sweep 1: last visible key of this row, relative to the tile
          const float* ncp = SWEEP == 2 ? nc + (p == 0 ? 0 : cols0) : nullptr;
          if (SWEEP == 1 && kSets == 2 && 2 * set >= n_ch) {  // this set has no columns in the part (never: a part of sweep 1 is 128 columns)
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(ebar);
          }
          if constexpr (SWEEP == 2 && kSets == 2) {
            // the sets take the leading and the trailing chunks of the two parts of a tile in turn: with 112 columns a
            // part that is 64 against 48 columns, and evens out over the tile
            switch (cols) {  // the shapes of a launch: one or two of these
#define AKV_COLS_CASE(C)                                                                          \
  case C:                                                                                         \
    if ((set ^ p) == 0) colsum_cols_set<C, 0>(taddr, ncp, sl2, ebar, lane, ra, a0, a1, a2, a3);   \
    else colsum_cols_set<C, 1>(taddr, ncp, sl2, ebar, lane, ra, a0, a1, a2, a3);                  \
    break;
              AKV_COLS_CASE(16) AKV_COLS_CASE(32) AKV_COLS_CASE(48) AKV_COLS_CASE(64)
              AKV_COLS_CASE(80) AKV_COLS_CASE(96) AKV_COLS_CASE(112) AKV_COLS_CASE(128)
#undef AKV_COLS_CASE
              default: break;  // r_pad is a multiple of 16 and a part at most 128 columns
            }
          } else {
          // one set: both steps of the part, unrolled; two sets: each takes one step (one copy of the code)
#pragma unroll
          for (int i = 0; i < (kSets == 2 ? 1 : 2); ++i) {
            const int st = kSets == 2 ? set : i;
            const int c0 = 2 * st;  // first chunk of 32 columns of this step
            if (c0 < n_ch) {
              const bool has_b = c0 + 1 < n_ch;
              const bool a_half = tail && c0 == n_ch - 1, b_half = tail && c0 + 1 == n_ch - 1;
              if (a_half) tmem_ld16_issue_lo(taddr + c0 * 32, ra);
              else tmem_ld32_issue(taddr + c0 * 32, ra);
              if (has_b) {
                if (b_half) tmem_ld16_issue_lo(taddr + (c0 + 1) * 32, rb);
                else tmem_ld32_issue(taddr + (c0 + 1) * 32, rb);
              }
              if (a_half) tmem_wait_lo(ra);
              else tmem_wait(ra);
              if (has_b) {
                if (b_half) tmem_wait_lo(rb);
                else tmem_wait(rb);
              }
              if (kSets == 2 || c0 + 2 >= n_ch) {  // this warp's columns of the part are in registers: its buffer goes back
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(ebar);
              }
              if constexpr (SWEEP == 1) {
                if (live) stats_step(ra, rb, masked, c0 * 32, last_col, sl, inv_sl, m_ref[p], Z[p]);  // padding rows only load
                __syncwarp();  // a warp may hold live and padding rows: rejoin before the warp-wide TMEM instructions
              } else {
                if (a_half) colsum_part<16>(ra, ncp + c0 * 32, sl2, a0, a1, a2, a3);
                else colsum_part<32>(ra, ncp + c0 * 32, sl2, a0, a1, a2, a3);
                if (has_b) {
                  if (b_half) colsum_part<16>(rb, ncp + (c0 + 1) * 32, sl2, a0, a1, a2, a3);
                  else colsum_part<32>(rb, ncp + (c0 + 1) * 32, sl2, a0, a1, a2, a3);
                }
              }
            }
          }
          }  // general loop
        }
        if (!ok) break;
        if (SWEEP == 2) {
          // The sets of a group (and the chunks of a window scored in several chunks) hold sums over different rows
          // of the same key: each adds its own into the score buffer, which sweep 1 cleared. With two addends the
          // result does not depend on their order.
          const int key = kt + gl;
          if (key < U.P) {
            const float sum = hsum(a0, a1, a2, a3);
            if (a.accumulate) atomicAdd(a.scores + U.score_base + key, sum);
            else a.scores[U.score_base + key] = sum;
          }
        }
      }
      if (!ok) break;
      if (SWEEP == 1) {
        // this group's share of the run (every second tile): one entry per row, merged by sweep 2 with the other
        // group's and the other parts'; a group without a tile in the run writes an empty entry
        float2* out = a.stats + ((static_cast<int64_t>(U.u) * a.max_parts + U.part) * kStatSets + g * kSets + set) * Rt + U.w0 * G;
#pragma unroll
        for (int p = 0; p < 2; ++p)
          if (p < n_parts && p * 128 + gl < live_rows) out[p * 128 + gl] = make_float2(m_ref[p], Z[p]);
      }
    }
  }

  // ---- teardown ----
  if (SWEEP == 1 && a.beside) chain_wait();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && sm->abort) atomicExch(a.status, AUDIOKV_ETIMEOUT);
  if (warp == kProducerWarp) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---- host side ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess ||
        qr != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Byte strides of the outer dimensions; a dimension of extent 1 takes a harmless stride when the
// caller's is zero. Returns false for a stride the copy engine cannot express.
bool fill_strides(int rank, const cuuint64_t* dims, const int64_t* elem_strides, cuuint64_t* out) {
  for (int i = 1; i < rank; ++i) {
    int64_t s = elem_strides[i - 1] * 2;
    if (dims[i] == 1 && s <= 0) s = 16;
    if (s <= 0 || (s & 15) || s >= (static_cast<int64_t>(1) << 40)) return false;
    out[i - 1] = static_cast<cuuint64_t>(s);
  }
  return true;
}

template <int SWEEP, int D, int CAP>
cudaError_t launch_sweep(const TmapPack<CAP>& tm, const UmmaArgs& args, int grid, size_t smem, cudaStream_t stream) {
  auto kern = score_umma_kernel<SWEEP, D, CAP>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  return launch_chained(kern, dim3(grid), dim3(n_threads(SWEEP)), smem, stream, tm, args);
}

template <int CAP>
cudaError_t launch_score_umma_cap(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* d_units, const int32_t* d_cta,
                                  const ScoreSchedule& sc, int slot, const void* q, const void* k, float* scores,
                                  float2* stats_ws, int max_parts, int* status, Launch ln, ScoreMapCache* cache,
                                  uint64_t plan_id, bool beside);

}  // namespace

int score_window_chunk(const Shape& sh) {
  if (sh.group < 1 || sh.window < 1) return 0;
  const int stage = kTileKeys * sh.head_dim * 2;
  for (int q_rows = 256; q_rows >= 128; q_rows -= 128) {
    const int room = kSmemLimit - 1024 - static_cast<int>(sizeof(Small)) - q_rows * sh.head_dim * 2;
    if (room < 2 * stage) continue;  // the K ring needs two stages
    const int w_max = q_rows / sh.group;
    if (w_max < 1) return 0;
    if (w_max >= sh.window) return sh.window;
    const int n_chunks = (sh.window + w_max - 1) / w_max;
    return (sh.window + n_chunks - 1) / n_chunks;  // chunks of equal size (the last one may be shorter)
  }
  return 0;
}

static std::atomic<long long> g_wait_cycles{kWaitCycles};
long long score_wait_cycles() { return g_wait_cycles.load(); }
void set_score_wait_cycles(long long cycles) { g_wait_cycles.store(cycles > 0 ? cycles : kWaitCycles); }

bool score_umma_takes(const Shape& sh) {
  if (sh.dtype != AUDIOKV_BF16) return false;
  const int wc = score_window_chunk(sh);
  return wc >= 1 && wc <= 256 && sh.group <= 256;
}

int score_stat_sets() { return kStatSets; }

int score_map_chunk(int n_req) { return n_req <= kMapChunkSmall ? kMapChunkSmall : kMapChunkLarge; }

cudaError_t launch_score_umma(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* d_units, const int32_t* d_cta,
                              const ScoreSchedule* scheds, int n_sched, const void* q, const void* k, float* scores,
                              float2* stats_ws, int max_parts, int* status, Launch ln, int head_begin, int head_end,
                              ScoreMapCache* cache, uint64_t plan_id, bool beside) {
  if (!score_umma_takes(sh)) return cudaErrorNotSupported;
  // every schedule that covers whole requests, in order; or the one schedule made for this range of heads
  bool any = false, any_before = false;  // only the first launch follows the caller's kernel
  for (int i = 0; i < n_sched; ++i) {
    const ScoreSchedule& sc = scheds[i];
    if (head_end < 0 ? !sc.whole_requests : (sc.whole_requests || sc.head_begin != head_begin || sc.head_end != head_end))
      continue;
    any = true;
    // the maps of a head range are those of its (single) request: slot 0; whole-request schedules come one per slot
    const int slot = sc.whole_requests ? sc.r_begin / score_map_chunk(sh.n_req) : 0;
    cudaError_t e = sh.n_req <= kMapChunkSmall
                        ? launch_score_umma_cap<kMapChunkSmall>(sh, h_reqs, d_units, d_cta, sc, slot, q, k, scores, stats_ws,
                                                                max_parts, status, ln, cache, plan_id, beside && !any_before)
                        : launch_score_umma_cap<kMapChunkLarge>(sh, h_reqs, d_units, d_cta, sc, slot, q, k, scores, stats_ws,
                                                                max_parts, status, ln, cache, plan_id, beside && !any_before);
    any_before = true;
    if (e != cudaSuccess) return e;
  }
  return any ? cudaSuccess : cudaErrorInvalidValue;
}

namespace {

template <int CAP>
cudaError_t launch_score_umma_cap(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* d_units, const int32_t* d_cta,
                                  const ScoreSchedule& sc, int slot, const void* q, const void* k, float* scores,
                                  float2* stats_ws, int max_parts, int* status, Launch ln, ScoreMapCache* cache,
                                  uint64_t plan_id, bool beside) {
  using Pack = TmapPack<CAP>;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int w_chunk = score_window_chunk(sh);
  const int R = w_chunk * sh.group, d = sh.head_dim;  // query rows of one Q tile

  UmmaArgs args{};
  args.sh = sh;
  args.stats = stats_ws;
  args.scores = scores;
  args.status = status;
  args.max_parts = max_parts;
  args.q_rows = R > 128 ? 256 : 128;
  args.r_pad = (R + 15) / 16 * 16;
  args.w_chunk = w_chunk;
  args.accumulate = (w_chunk < sh.window || epi_sets(2) > 1) ? 1 : 0;
  args.beside = beside ? 1 : 0;
  args.wait_cycles = score_wait_cycles();
  const int q_bytes = args.q_rows * d * 2, stage = kTileKeys * d * 2;
  const int room = kSmemLimit - 1024 - static_cast<int>(sizeof(Small)) - q_bytes;
  args.n_stages = room / stage < kMaxStages ? room / stage : kMaxStages;
  const size_t smem = 1024 + static_cast<size_t>(q_bytes) + static_cast<size_t>(args.n_stages) * stage + sizeof(Small);

  // Tensor maps are kernel arguments, CAP requests' worth per launch: one pack per run of CAP requests. They depend
  // on the buffers, the request table and the strides: the same buffers under the same plan reuse them.
  const int n_slots = (sh.n_req + CAP - 1) / CAP;
  std::vector<unsigned char> local;
  std::vector<unsigned char>& packs = cache ? cache->packs : local;
  const size_t pack_bytes = sizeof(Pack) * static_cast<size_t>(n_slots) + 64;  // + room to align to 64 bytes
  const bool same = cache && cache->q == q && cache->k == k && cache->plan_id == plan_id &&
                    cache->page_size == sh.page_size && packs.size() == pack_bytes &&
                    cache->encoded.size() == static_cast<size_t>(n_slots);
  if (!same) {
    packs.assign(pack_bytes, 0);
    if (cache) {
      cache->encoded.assign(n_slots, 0);
      cache->q = q;
      cache->k = k;
      cache->plan_id = plan_id;
      cache->page_size = sh.page_size;
    }
  }
  unsigned char* pack0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(packs.data()) + 63) & ~uintptr_t(63));
  Pack& tm = *reinterpret_cast<Pack*>(pack0 + sizeof(Pack) * static_cast<size_t>(slot));
  const int r0 = slot * CAP, r1 = r0 + CAP < sh.n_req ? r0 + CAP : sh.n_req;
  if (!(cache && cache->encoded[slot])) {
    for (int r = r0; r < r1; ++r) {
      {
        const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(sh.n_q_heads),
                                    static_cast<cuuint64_t>(sh.window), static_cast<cuuint64_t>(sh.n_layers)};
        const int64_t es[3] = {sh.q_stride_head, sh.q_stride_tok, sh.q_stride_layer};
        cuuint64_t strides[3];
        if (!fill_strides(4, dims, es, strides)) return cudaErrorNotSupported;
        const cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(sh.group), static_cast<cuuint32_t>(w_chunk), 1u};
        const cuuint32_t ones[4] = {1u, 1u, 1u, 1u};
        void* base = const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(q) + h_reqs[r].q_offset);
        if (enc(&tm.q[r - r0], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, ones,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
          return cudaErrorNotSupported;
      }
      if (sh.page_size != 0 && r > r0) continue;  // one map of the whole pool serves every request
      const bool paged = sh.page_size != 0;
      const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d),
                                  paged ? static_cast<cuuint64_t>(sh.n_pages) * sh.page_size
                                        : static_cast<cuuint64_t>(h_reqs[r].L),
                                  static_cast<cuuint64_t>(sh.n_kv_heads), static_cast<cuuint64_t>(sh.n_layers)};
      const int64_t es[3] = {sh.kv_stride_tok, sh.kv_stride_head, sh.kv_stride_layer};
      cuuint64_t strides[3];
      if (!fill_strides(4, dims, es, strides)) return cudaErrorNotSupported;
      const cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(paged ? sh.page_size : kTileKeys), 1u, 1u};
      const cuuint32_t ones[4] = {1u, 1u, 1u, 1u};
      void* base = const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(k) + (paged ? 0 : h_reqs[r].kv_offset));
      if (enc(&tm.k[r - r0], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorNotSupported;
    }
    if (cache) cache->encoded[slot] = 1;
  }
  args.r0 = r0;
  cudaError_t e;
#define AKV_SWEEP(SW, DD)                                                              \
  args.units = d_units + sc.unit_off[SW - 1];                                          \
  args.cta_begin = d_cta + sc.cta_off[SW - 1];                                         \
  if (sc.grid[SW - 1] > 0) {                                                           \
    e = launch_sweep<SW, DD>(tm, args, sc.grid[SW - 1], smem, ln.stream);              \
    if (e != cudaSuccess) return e;                                                    \
    ln.done(SW == 1 ? "score_umma_stats" : "score_umma_colsum");                      \
  }
  if (d == 64) {
    AKV_SWEEP(1, 64);
    AKV_SWEEP(2, 64);
  } else if (d == 128) {
    AKV_SWEEP(1, 128);
    AKV_SWEEP(2, 128);
  } else {
    AKV_SWEEP(1, 256);
    AKV_SWEEP(2, 256);
  }
#undef AKV_SWEEP
  return cudaSuccess;
}

}  // namespace

}  // namespace akv
