// Importance scores for bf16 inputs on the tcgen05 tensor cores (sm_100a).
//
// The score of key j is the sum, over the W window rows and the G query heads of a KV
// head, of softmax probabilities. A column sum mixes rows with different normalisers,
// so the keys are swept twice:
//   sweep 1  D[row][key]  = Q K^T  (query rows on the TMEM lanes): every thread owns one
//            row and keeps its running maximum and sum of exp2 over the keys of a slab;
//            one (max, sum) pair per (head, slab, row) goes to the statistics buffer.
//   sweep 2  D[key][row]  = K Q^T  (keys on the TMEM lanes): every thread owns one key
//            and adds exp2(z - max - log2 sum) over the rows; no cross-thread reduction.
// Both sweeps are one persistent kernel (one CTA per SM) with three roles:
//   warp 16   TMA producer: the Q tile of a head once, K tiles of 128 keys through a ring;
//   warp 17   MMA issuer: tcgen05.mma, bf16 x bf16 -> fp32 in TMEM, two accumulator buffers;
//   warps 0-15 four groups of 128 threads that read the accumulators (tcgen05.ld) and do the
//             softmax arithmetic.
// Q and K tiles are K-major with the 128-byte swizzle, so the same shared-memory tile is
// the A operand of one sweep and the B operand of the other.
// Every wait on an mbarrier is bounded: when one runs out the CTA stops, the kernel
// writes AUDIOKV_ETIMEOUT to the status word and returns with its TMEM released.
#include <cuda.h>
#include <stddef.h>

#include "common.cuh"

namespace akv {
namespace {

constexpr int kTileKeys = 128;    // keys per K tile (UMMA M in sweep 2, N in sweep 1)
constexpr int kEpiWarps = 16;      // four epilogue groups of four warps (one warp per TMEM lane quarter)
constexpr int kProducerWarp = kEpiWarps;
constexpr int kMmaWarp = kEpiWarps + 1;
constexpr int kThreads = (kEpiWarps + 2) * 32;
constexpr int kAccCols = 256;     // TMEM columns of one accumulator buffer
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxStages = 8;
constexpr long long kWaitCycles = 2000000000LL;  // about one second
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
  const ScoreUnit* units;  // this sweep's schedule, in processing order
  float2* stats;
  float* scores;
  int* status;
  int n_slab;     // slabs per head in the statistics buffer
  int slab_keys;  // keys per slab, a multiple of kTileKeys
  int n_units;    // (head, slab) units of this sweep
  int q_rows;     // rows of the Q tile in shared memory: 128 or 256
  int r_pad;      // W * G rounded up to 16
  int n_stages;   // K ring depth
  int r0;         // first request of this launch: request r uses maps q[r - r0], k[r - r0]
};

struct Small {
  alignas(16) float negc[2][256];     // sweep 2: -(max + log2 sum) per row, by head parity (read 16 bytes at a time)
  alignas(16) float2 mrg[2][3][128];  // sweep 1: partial statistics of the groups that share a row, by unit parity
  alignas(16) float part[4][3][128];  // sweep 2: partial column sums of groups 1-3, by tile number mod 4
  alignas(8) uint64_t k_full[kMaxStages];
  uint64_t k_empty[kMaxStages];
  uint64_t q_full, q_empty;
  uint64_t acc_full[2][2], acc_empty[2][2];  // [group][buffer]: each epilogue group has its own accumulator stream
  uint64_t all_bar;     // all epilogue threads (512 arrivals)
  uint64_t part_full[4];  // sweep 2: the twelve warps of groups 1-3 have written part[i]
  uint64_t drain;       // stop path only: the MMAs still in flight
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
// Bounded wait. Returns false when the CTA is stopping (this or another wait ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort,
                                          long long limit = kWaitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0) {
      if (*abort) return false;
      if (clock64() - t0 > limit) {
        *abort = 1;
        return false;
      }
    }
  }
  return true;
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

// Sweep 1: N = NH * 32 logits of this thread's row (columns col0 .. col0 + N - 1 of the tile). Updates the
// row's running maximum (raw dot products) and its sum of exp2 relative to that maximum.
template <int NH>
__device__ __forceinline__ void stats_part(uint32_t (&r)[NH][32], bool masked, int col0, int last_col, float sl,
                                           float& m_run, float& Z) {
  constexpr int N = NH * 32;
  if (masked) {
#pragma unroll
    for (int i = 0; i < N; ++i)
      if (col0 + i > last_col) r[i >> 5][i & 31] = 0xff800000u;  // -inf
  }
  float cm = __uint_as_float(r[0][0]);
#pragma unroll
  for (int i = 1; i + 1 < N; i += 2)
    cm = max3(cm, __uint_as_float(r[i >> 5][i & 31]), __uint_as_float(r[(i + 1) >> 5][(i + 1) & 31]));
  cm = fmaxf(cm, __uint_as_float(r[NH - 1][31]));
  if (cm == -INFINITY) return;  // fully masked: adds nothing
  const float m_new = fmaxf(m_run, cm);
  const float rescale = ex2((m_run - m_new) * sl);  // first time: exp2(-inf) = 0
  m_run = m_new;
  const float nb = -m_new * sl;
  const f32x2 sl2 = pack2(sl, sl), nb2 = pack2(nb, nb);
  f32x2 a0 = pack2(0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;
#pragma unroll
  for (int i = 0; i < N; i += 8) {
    a0 = add2(a0, ex2_2(fma2(pack2(r[i >> 5][i & 31], r[i >> 5][(i & 31) + 1]), sl2, nb2)));
    a1 = add2(a1, ex2_2(fma2(pack2(r[i >> 5][(i & 31) + 2], r[i >> 5][(i & 31) + 3]), sl2, nb2)));
    a2 = add2(a2, ex2_2(fma2(pack2(r[i >> 5][(i & 31) + 4], r[i >> 5][(i & 31) + 5]), sl2, nb2)));
    a3 = add2(a3, ex2_2(fma2(pack2(r[i >> 5][(i & 31) + 6], r[i >> 5][(i & 31) + 7]), sl2, nb2)));
  }
  Z = fmaf(Z, rescale, hsum(a0, a1, a2, a3));
}
// One tile of sweep 1, NCH chunks of 32 columns: the next chunk's TMEM load runs under the arithmetic of this one.
template <int NCH>
__device__ __forceinline__ void stats_tile(uint32_t taddr, bool live, bool masked, int col0, int last_col, float sl,
                                           float& m_run, float& Z) {
  uint32_t ra[1][32], rb[1][32];
  tmem_ld32_issue(taddr, ra[0]);
#pragma unroll
  for (int c = 0; c < NCH; c += 2) {
    tmem_wait(ra[0]);
    if (c + 1 < NCH) tmem_ld32_issue(taddr + (c + 1) * 32, rb[0]);
    if (live) stats_part<1>(ra, masked, col0 + c * 32, last_col, sl, m_run, Z);  // padding rows only take part in the loads
    __syncwarp();  // a warp may hold live and padding rows: rejoin before the warp-wide TMEM instructions
    if (c + 1 < NCH) {
      tmem_wait(rb[0]);
      if (c + 2 < NCH) tmem_ld32_issue(taddr + (c + 2) * 32, ra[0]);
      if (live) stats_part<1>(rb, masked, col0 + (c + 1) * 32, last_col, sl, m_run, Z);
      __syncwarp();
    }
  }
}

// Sweep 2: N logits of this thread's key against N query rows; nc = their -(max + log2 sum), 16-byte aligned.
// Adds exp2(z * sl + nc[row]) into four pairs of partial sums.
template <int N>
__device__ __forceinline__ void colsum_part(const uint32_t (&r)[N], const float* __restrict__ nc, f32x2 sl2, f32x2& a0,
                                            f32x2& a1, f32x2& a2, f32x2& a3) {
  const ulonglong2* nc2 = reinterpret_cast<const ulonglong2*>(nc);
#pragma unroll
  for (int j = 0; j < N; j += 8) {
    const ulonglong2 v = nc2[j >> 2], w = nc2[(j >> 2) + 1];
    a0 = add2(a0, ex2_2(fma2(pack2(r[j], r[j + 1]), sl2, v.x)));
    a1 = add2(a1, ex2_2(fma2(pack2(r[j + 2], r[j + 3]), sl2, v.y)));
    a2 = add2(a2, ex2_2(fma2(pack2(r[j + 4], r[j + 5]), sl2, w.x)));
    a3 = add2(a3, ex2_2(fma2(pack2(r[j + 6], r[j + 7]), sl2, w.y)));
  }
}
// One tile of sweep 2: this group's n_u (<= 4) units of 16 TMEM columns starting at taddr; nc points at the
// first of its query rows. Chunks of 32 columns and a last one of 16; the other warps of the scheduler cover
// the load latency.
__device__ __forceinline__ float colsum_tile(uint32_t taddr, int n_u, const float* __restrict__ nc, float sl) {
  const int n32 = n_u >> 1;
  const bool tail = (n_u & 1) != 0;
  uint32_t ra[32], rt[16];
  if (tail) tmem_ld16_issue(taddr + n32 * 32, rt);
  const f32x2 sl2 = pack2(sl, sl);
  f32x2 a0 = pack2(0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    if (c < n32) {
      tmem_ld32_issue(taddr + c * 32, ra);
      tmem_wait(ra);
      colsum_part<32>(ra, nc + c * 32, sl2, a0, a1, a2, a3);
    }
  }
  if (tail) {
    tmem_wait(rt);
    colsum_part<16>(rt, nc + n32 * 32, sl2, a0, a1, a2, a3);
  }
  return hsum(a0, a1, a2, a3);
}

template <int SWEEP, int D, int CAP>
__global__ void __launch_bounds__(kThreads, 1)
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
  const int R = sh.window * sh.group, G = sh.group;
  const bool both = SWEEP == 1 && R > 128;   // sweep 1 with two row blocks: each group reads its own block of every tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = a.n_stages;

  // ---- set-up ----
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(smem_u32(&sm->k_full[s]), 1);
      mbar_init(smem_u32(&sm->k_empty[s]), 1);
    }
    mbar_init(smem_u32(&sm->q_full), 1);
    mbar_init(smem_u32(&sm->q_empty), 1);
    for (int g = 0; g < 2; ++g) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(smem_u32(&sm->acc_full[g][b]), 1);
        mbar_init(smem_u32(&sm->acc_empty[g][b]), 8);  // the two epilogue groups that share the stream
      }
    }
    mbar_init(smem_u32(&sm->all_bar), kEpiWarps * 32);
    for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&sm->part_full[i]), 12);
    mbar_init(smem_u32(&sm->drain), 1);
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
  if (SWEEP == 1) chain_wait();
  chain_release();
  const uint32_t tmem_base = sm->tmem_base;

  const int unit_begin = static_cast<int>(static_cast<int64_t>(blockIdx.x) * a.n_units / gridDim.x);
  const int unit_end = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * a.n_units / gridDim.x);

  // Every tile is split between the two epilogue groups, and each group gets its share through its own
  // pair of accumulator buffers (TMEM columns (2 b + g) * 128 ..), filled by its own MMAs: the groups
  // then run half a tile apart instead of in step, and one group's exponentials cover the other's
  // loads and maxima.
  //   sweep 1, two row blocks: group g = row block g, all 128 keys;
  //   sweep 1, one row block:  group g = keys 64 g .. 64 g + 63 of every row;
  //   sweep 2: group 0 = the first half of the query rows (in units of 16), group 1 = the rest.
  const int n16 = a.r_pad >> 4, u_split = (n16 + 1) >> 1;
  auto share_units = [&](int g) { return g == 0 ? u_split : n16 - u_split; };  // sweep 2: units of 16 rows

  if (warp == kProducerWarp) {
    // ---- TMA producer ----
    // Lane 0 runs the ring. With a paged pool the 128 / page_size pages of a tile are fetched by as many lanes,
    // one page each (a copy costs its issuing thread about a hundred cycles, and a tile of 16-token pages is 8 to 32
    // copies): those lanes walk the same schedule, lane 0 alone waits and arms the barriers, and its result reaches
    // the others through the shuffle that also orders their copies after the arming.
    const int n_sub = a.sh.page_size ? kTileKeys >> a.sh.page_shift : 1;
    const uint32_t lanes = (1u << n_sub) - 1u;
    if (lane < n_sub) {
      // Sweep 2 is the last reader of K before the gather: its tiles are marked evict-first in L2, so that what the
      // next kernels need (scores, tables, their code) is not pushed out by the stream (measured: 0.7 % of the pass)
      const uint64_t evict_first = l2_evict_first();
      int it = 0, heads = 0, prev_u = -1, s = 0;  // s, ph: slot of the K ring and its phase
      uint32_t ph = 0;
      bool ok = true;
      ScoreUnit Unext = a.units[unit_begin < unit_end ? unit_begin : 0];
      for (int n = unit_begin; n < unit_end && ok; ++n) {
        const ScoreUnit U = Unext;
        if (n + 1 < unit_end) Unext = a.units[n + 1];  // the next descriptor arrives under this unit's work
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
            if (t == 0 && U.u != prev_u) {
              if (heads > 0) mine = mbar_wait(smem_u32(&sm->q_empty), (heads - 1) & 1, abort);  // MMAs on the old Q are done
              if (mine) {
                const uint32_t qbar = smem_u32(&sm->q_full);
                mbar_expect_tx(qbar, static_cast<uint32_t>(R) * D * 2);
                for (int kb = 0; kb < KB; ++kb)
                  tma_load_4d(smem_u32(q_s + kb * q_blk), &tm.q[U.r - a.r0], qbar, kb * 64, U.h * G, 0, U.l);
                prev_u = U.u;
                ++heads;
              }
            }
            if (mine) mine = mbar_wait(smem_u32(&sm->k_empty[s]), ph ^ 1, abort);
            if (mine) mbar_expect_tx(bar, kKStage);
          }
          ok = __shfl_sync(lanes, mine, 0);
          if (!ok) break;
          if (a.sh.page_size == 0) {
            for (int kb = 0; kb < KB; ++kb) {
              if (SWEEP == 2)
                tma_load_4d_hint(smem_u32(k_s + s * kKStage + kb * kKBlk), &tm.k[U.r - a.r0], bar, kb * 64,
                                 U.kt0 + t * kTileKeys, U.h, U.l, evict_first);
              else
                tma_load_4d(smem_u32(k_s + s * kKStage + kb * kKBlk), &tm.k[U.r - a.r0], bar, kb * 64,
                            U.kt0 + t * kTileKeys, U.h, U.l);
            }
          } else {
            // k[0] maps the whole pool as (d, page * page_size + token in page, KV head, layer) with a box of one
            // page: at least 16 rows of 128 bytes, whole swizzle groups, so the tile comes out as in the contiguous case
            for (int kb = 0; kb < KB; ++kb) {
              const uint32_t dst = smem_u32(k_s + s * kKStage + kb * kKBlk + lane * a.sh.page_size * 128);
              if (SWEEP == 2) tma_load_4d_hint(dst, &tm.k[0], bar, kb * 64, page_y, U.h, U.l, evict_first);
              else tma_load_4d(dst, &tm.k[0], bar, kb * 64, page_y, U.h, U.l);
            }
          }
          if (++s == S) {
            s = 0;
            ph ^= 1;
          }
        }
      }
      if (lane == 0 && *abort) {  // let the copies still in flight land before the CTA goes away
        const long long short_limit = 200000000LL;
        for (int j = it > S ? it - S : 0; j < it; ++j)
          mbar_wait(smem_u32(&sm->k_full[j % S]), (j / S) & 1, abort, short_limit);
        if (heads > 0) mbar_wait(smem_u32(&sm->q_full), (heads - 1) & 1, abort, short_limit);
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      // ---- MMA issuer ----
      int it = 0, heads = 0, prev_u = -1, s = 0;
      uint32_t ph = 0;
      bool ok = true;
      const uint32_t idesc1 = both ? umma_idesc(128, kTileKeys) : umma_idesc(128, kTileKeys / 2);
      ScoreUnit Unext = a.units[unit_begin < unit_end ? unit_begin : 0];
      for (int n = unit_begin; n < unit_end && ok; ++n) {
        const ScoreUnit U = Unext;
        if (n + 1 < unit_end) Unext = a.units[n + 1];  // the next descriptor arrives under this unit's work
        if (U.u != prev_u) {
          if (prev_u != -1) umma_commit(smem_u32(&sm->q_empty));
          ok = mbar_wait(smem_u32(&sm->q_full), heads & 1, abort);
          if (!ok) break;
          tc_fence_after();
          prev_u = U.u;
          ++heads;
        }
        for (int t = 0; t < U.n_tiles && ok; ++t, ++it) {
          ok = mbar_wait(smem_u32(&sm->k_full[s]), ph, abort);
          if (!ok) break;
          const int b = it & 1;
          const uint32_t k_addr = smem_u32(k_s + s * kKStage);
          const uint32_t q_addr = smem_u32(q_s);
          for (int g = 0; g < 2; ++g) {
            if (SWEEP == 2 && share_units(g) == 0) continue;
            ok = mbar_wait(smem_u32(&sm->acc_empty[g][b]), ((it >> 1) & 1) ^ 1, abort);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (2 * b + g) * 128;
            // byte offsets of the group's share inside the Q tile / the K tile (multiples of 1024: whole 8-row groups)
            const uint32_t q_off = SWEEP == 1 ? (both ? g * (128 * 128) : 0) : (g == 0 ? 0 : u_split * 16 * 128);
            const uint32_t k_off = SWEEP == 1 && !both ? g * (64 * 128) : 0;
            const uint32_t idesc = SWEEP == 1 ? idesc1 : umma_idesc(kTileKeys, share_units(g) * 16);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
              for (int ks = 0; ks < 4; ++ks) {
                const uint64_t dq = umma_desc(q_addr + kb * q_blk + q_off + ks * 32);
                const uint64_t dk = umma_desc(k_addr + kb * kKBlk + k_off + ks * 32);
                if (SWEEP == 1) umma_bf16(d_tmem, dq, dk, idesc, (kb | ks) != 0);
                else umma_bf16(d_tmem, dk, dq, idesc, (kb | ks) != 0);
              }
            }
            umma_commit(smem_u32(&sm->acc_full[g][b]));
          }
          umma_commit(smem_u32(&sm->k_empty[s]));
          if (++s == S) {
            s = 0;
            ph ^= 1;
          }
        }
      }
      if (*abort) {  // TMEM must not be released under MMAs that are still running
        umma_commit(smem_u32(&sm->drain));
        mbar_wait(smem_u32(&sm->drain), 0, abort, 200000000LL);
      }
    }
  } else {
    // ---- epilogue: four groups of four warps; warp w reads TMEM lanes 32 (w % 4) .. +31 ----
    // Groups 2 st and 2 st + 1 share accumulator stream st and split its columns in two:
    //   sweep 1, two row blocks: stream = row block, group = 64 of its 128 key columns;
    //   sweep 1, one row block:  stream = 64 key columns, group = 32 of them;
    //   sweep 2: stream = half of the query rows (units of 16), group = half of those; groups 1-3 hand their
    //            partial column sums to group 0 through shared memory.
    // Four warps per scheduler keep the special-function unit fed while others load, reduce or wait.
    const int g4 = warp >> 2, quarter = warp & 3;
    const int st = g4 >> 1, sub = g4 & 1;
    const int gl = quarter * 32 + lane;  // thread index inside the group = TMEM lane
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const float sl = sh.scale_log2e;
    int it = 0, prev_u = -1, n_done = 0, heads = 0;
    uint32_t all_phase = 0;
    bool ok = true;
    const int row = (both ? st * 128 : 0) + gl;                // sweep 1: this thread's query row
    const int col0 = both ? sub * 64 : st * 64 + sub * 32;     // sweep 1: first key column (of the tile) of its share
    const int tcol1 = both ? sub * 64 : sub * 32;              // ... and that column inside the stream's accumulator
    const int win_i = row / G;                                 // window row of that query row
    const bool live = row < R;
    // sweep 2: the stream's units of 16 query rows, and this group's part of them
    const int st_u0 = st == 0 ? 0 : u_split, st_n = share_units(st);
    const int half_n = (st_n + 1) >> 1;
    const int my_u0 = sub == 0 ? 0 : half_n, my_n = sub == 0 ? half_n : st_n - half_n;
    if (SWEEP == 2) chain_wait();  // the statistics of sweep 1 are complete and visible
    ScoreUnit Unext = a.units[unit_begin < unit_end ? unit_begin : 0];
    for (int n = unit_begin; n < unit_end && ok; ++n, ++n_done) {
      const ScoreUnit U = Unext;
      if (n + 1 < unit_end) Unext = a.units[n + 1];
      if (SWEEP == 2 && U.u != prev_u) {
        // Merge the slabs' statistics of this head: negc[row] = -(max + log2 sum); padding rows get -inf.
        // One row per thread of the first two groups, eight independent loads in flight at a time.
        const int slabs = U.head_slabs;
        const int rr = g4 * 128 + gl;
        if (rr < 256) {
          float c = -INFINITY;
          if (rr < R) {
            const float2* hs = a.stats + static_cast<int64_t>(U.u) * a.n_slab * R + rr;
            float M = -INFINITY, Zt = 0.f;
            for (int s0 = 0; s0 < slabs; s0 += 8) {
              float2 sv[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                sv[i] = s0 + i < slabs ? __ldg(hs + static_cast<int64_t>(s0 + i) * R) : make_float2(-INFINITY, 0.f);
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
          // two copies by head parity: a slower warp may still read the previous head's
          sm->negc[heads & 1][rr] = c;
        }
        ++heads;
        mbar_arrive(smem_u32(&sm->all_bar));
        ok = mbar_wait(smem_u32(&sm->all_bar), all_phase, abort);
        all_phase ^= 1;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      prev_u = U.u;
      float m_run = -INFINITY, Z = 0.f;  // sweep 1: this thread's row (its share of the columns)
      for (int t = 0; t < U.n_tiles; ++t, ++it) {
        const int b = it & 1;
        const bool stream_on = SWEEP == 1 || st_n > 0;  // the MMA thread skips a stream without rows
        if (stream_on) {
          ok = mbar_wait(smem_u32(&sm->acc_full[st][b]), (it >> 1) & 1, abort);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        const int kt = U.kt0 + t * kTileKeys;
        const uint32_t taddr = lane_addr + (2 * b + st) * 128;
        if (SWEEP == 1) {
          const bool masked = kt + kTileKeys - 1 > U.P;  // the tile reaches into the window: causal mask, end of request
          const int last_col = U.P + win_i - kt;         // last visible key of this row, relative to the tile
          if (both) stats_tile<2>(taddr + tcol1, live, masked, col0, last_col, sl, m_run, Z);
          else stats_tile<1>(taddr + tcol1, live, masked, col0, last_col, sl, m_run, Z);
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&sm->acc_empty[st][b]));
        } else {
          float acc = 0.f;
          if (stream_on) {
            if (my_n > 0) acc = colsum_tile(taddr + my_u0 * 16, my_n, sm->negc[(heads - 1) & 1] + (st_u0 + my_u0) * 16, sl);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->acc_empty[st][b]));
          }
          const int slot = it & 3;
          if (g4 != 0) {
            sm->part[slot][g4 - 1][gl] = acc;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->part_full[slot]));
          } else {
            // Slot it & 3 is written again four tiles on. By then the MMAs of tile it + 4 have been issued,
            // so this group has released the buffer of tile it + 2, which it does after the read below.
            ok = mbar_wait(smem_u32(&sm->part_full[slot]), (it >> 2) & 1, abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int key = kt + gl;
            if (key < U.P)
              a.scores[U.score_base + key] = (acc + sm->part[slot][0][gl]) + (sm->part[slot][1][gl] + sm->part[slot][2][gl]);
          }
        }
      }
      if (!ok) break;
      if (SWEEP == 1) {
        // the groups that share a row hand their statistics to the first of them
        float2* out = a.stats + (static_cast<int64_t>(U.u) * a.n_slab + U.slab) * R;
        float2(*mg)[128] = sm->mrg[n_done & 1];
        const bool writer = both ? sub == 0 : g4 == 0;
        if (!writer) mg[both ? st : g4 - 1][gl] = make_float2(m_run, Z);
        mbar_arrive(smem_u32(&sm->all_bar));
        ok = mbar_wait(smem_u32(&sm->all_bar), all_phase, abort);
        all_phase ^= 1;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (writer && live) {
          const int s0 = both ? st : 0, ns_ = both ? 1 : 3;
          float M = m_run;
          for (int o = 0; o < ns_; ++o) M = fmaxf(M, mg[s0 + o][gl].x);
          float Zt = Z > 0.f ? Z * ex2((m_run - M) * sl) : 0.f;
          for (int o = 0; o < ns_; ++o) {
            const float2 pz = mg[s0 + o][gl];
            if (pz.y > 0.f) Zt += pz.y * ex2((pz.x - M) * sl);
          }
          out[row] = make_float2(M * sl, Zt);
        }
      }
    }
  }

  // ---- teardown ----
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
  return launch_chained(kern, dim3(grid), dim3(kThreads), smem, stream, tm, args);
}

template <int CAP>
cudaError_t launch_score_umma_cap(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* units1, const int* unit_pre1,
                                  const ScoreUnit* units2, const int* unit_pre2, const void* q, const void* k,
                                  float* scores, float2* stats_ws, int n_slab, int slab_keys, int* status, Launch ln,
                                  int head_begin, int head_end, ScoreMapCache* cache, uint64_t plan_id);

}  // namespace

bool score_umma_takes(const Shape& sh) {
  if (sh.dtype != AUDIOKV_BF16) return false;
  const int R = sh.window * sh.group;
  if (R > 256 || sh.group > 256 || sh.window > 256) return false;
  const int q_rows = R > 128 ? 256 : 128;
  const int q_bytes = q_rows * sh.head_dim * 2, stage = kTileKeys * sh.head_dim * 2;
  const int room = kSmemLimit - 1024 - static_cast<int>(sizeof(Small)) - q_bytes;
  return room >= 2 * stage;
}

cudaError_t launch_score_umma(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* units1, const int* unit_pre1,
                              const ScoreUnit* units2, const int* unit_pre2, const void* q, const void* k,
                              float* scores, float2* stats_ws, int n_slab, int slab_keys, int* status, Launch ln,
                              int head_begin, int head_end, ScoreMapCache* cache, uint64_t plan_id) {
  if (sh.n_req <= kMapChunkSmall)
    return launch_score_umma_cap<kMapChunkSmall>(sh, h_reqs, units1, unit_pre1, units2, unit_pre2, q, k, scores, stats_ws,
                                                 n_slab, slab_keys, status, ln, head_begin, head_end, cache, plan_id);
  return launch_score_umma_cap<kMapChunkLarge>(sh, h_reqs, units1, unit_pre1, units2, unit_pre2, q, k, scores, stats_ws,
                                               n_slab, slab_keys, status, ln, head_begin, head_end, cache, plan_id);
}

namespace {

template <int CAP>
cudaError_t launch_score_umma_cap(const Shape& sh, const ReqDesc* h_reqs, const ScoreUnit* units1, const int* unit_pre1,
                                  const ScoreUnit* units2, const int* unit_pre2, const void* q, const void* k,
                                  float* scores, float2* stats_ws, int n_slab, int slab_keys, int* status, Launch ln,
                                  int head_begin, int head_end, ScoreMapCache* cache, uint64_t plan_id) {
  constexpr int kMapChunk = CAP;
  using Pack = TmapPack<CAP>;
  if (!score_umma_takes(sh) || slab_keys % kTileKeys) return cudaErrorNotSupported;
  if (head_end >= 0 && sh.n_req != 1) return cudaErrorInvalidValue;  // head ranges: one request only
  EncodeTiledFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int R = sh.window * sh.group, d = sh.head_dim;

  UmmaArgs args{};
  args.sh = sh;
  args.stats = stats_ws;
  args.scores = scores;
  args.status = status;
  args.n_slab = n_slab;
  args.slab_keys = slab_keys;
  args.q_rows = R > 128 ? 256 : 128;
  args.r_pad = (R + 15) / 16 * 16;
  const int q_bytes = args.q_rows * d * 2, stage = kTileKeys * d * 2;
  const int room = kSmemLimit - 1024 - static_cast<int>(sizeof(Small)) - q_bytes;
  args.n_stages = room / stage < kMaxStages ? room / stage : kMaxStages;
  const size_t smem = 1024 + static_cast<size_t>(q_bytes) + static_cast<size_t>(args.n_stages) * stage + sizeof(Small);

  int dev = 0, n_sm = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;

  // Tensor maps are kernel arguments, CAP requests' worth per launch: a longer batch takes both sweeps chunk
  // by chunk. Sweep 1 lists the units by ascending request, sweep 2 by descending request, so a chunk of requests
  // is one contiguous run of either list.
  const int n_units2 = unit_pre2[sh.n_req];
  const int n_chunks = (sh.n_req + kMapChunk - 1) / kMapChunk;
  // the maps depend on the buffers, the request table and the strides: the same buffers under the same plan reuse them
  std::vector<unsigned char> local;
  std::vector<unsigned char>& packs = cache ? cache->packs : local;
  const size_t pack_bytes = sizeof(Pack) * static_cast<size_t>(n_chunks) + 64;  // + room to align to 64 bytes
  const bool reuse = cache && cache->q == q && cache->k == k && cache->plan_id == plan_id &&
                     cache->page_size == sh.page_size && packs.size() == pack_bytes;
  if (!reuse) {
    if (cache) cache->q = nullptr;  // stays invalid if the encoding below fails half way
    packs.assign(pack_bytes, 0);
  }
  unsigned char* pack0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(packs.data()) + 63) & ~uintptr_t(63));
  for (int r0 = 0; r0 < sh.n_req; r0 += kMapChunk) {
    const int r1 = r0 + kMapChunk < sh.n_req ? r0 + kMapChunk : sh.n_req;
    Pack& tm = *reinterpret_cast<Pack*>(pack0 + sizeof(Pack) * static_cast<size_t>(r0 / kMapChunk));
    for (int r = r0; r < r1 && !reuse; ++r) {
      {
        const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(sh.n_q_heads),
                                    static_cast<cuuint64_t>(sh.window), static_cast<cuuint64_t>(sh.n_layers)};
        const int64_t es[3] = {sh.q_stride_head, sh.q_stride_tok, sh.q_stride_layer};
        cuuint64_t strides[3];
        if (!fill_strides(4, dims, es, strides)) return cudaErrorNotSupported;
        const cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(sh.group), static_cast<cuuint32_t>(sh.window), 1u};
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
    args.r0 = r0;
    const ScoreUnit* u1 = units1 + unit_pre1[r0];
    int n1 = unit_pre1[r1] - unit_pre1[r0];
    const ScoreUnit* u2 = units2 + (n_units2 - unit_pre2[r1]);
    int n2 = unit_pre2[r1] - unit_pre2[r0];
    if (head_end >= 0) {
      // one request: every head has the same number of slabs in a sweep, and its units are consecutive
      const int s1 = n1 / sh.heads_per_req, s2 = n2 / sh.heads_per_req;
      u1 += head_begin * s1;
      n1 = (head_end - head_begin) * s1;
      u2 += (sh.heads_per_req - head_end) * s2;  // sweep 2 lists the heads backwards
      n2 = (head_end - head_begin) * s2;
    }

#define AKV_SWEEP(SW, DD, UNITS, N)                                                  \
  args.n_units = (N);                                                                \
  args.units = (UNITS);                                                              \
  e = launch_sweep<SW, DD>(tm, args, (N) < n_sm ? (N) : n_sm, smem, ln.stream);      \
  if (e != cudaSuccess) return e;                                                    \
  ln.done(SW == 1 ? "score_umma_stats" : "score_umma_colsum")
    if (d == 64) {
      AKV_SWEEP(1, 64, u1, n1);
      AKV_SWEEP(2, 64, u2, n2);
    } else if (d == 128) {
      AKV_SWEEP(1, 128, u1, n1);
      AKV_SWEEP(2, 128, u2, n2);
    } else {
      AKV_SWEEP(1, 256, u1, n1);
      AKV_SWEEP(2, 256, u2, n2);
    }
#undef AKV_SWEEP
  }
  if (cache && !reuse) {
    cache->q = q;
    cache->k = k;
    cache->plan_id = plan_id;
    cache->page_size = sh.page_size;
  }
  return cudaSuccess;
}

}  // namespace

}  // namespace akv
