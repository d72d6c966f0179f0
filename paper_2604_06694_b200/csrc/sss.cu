// Spectral Score Smoothing: one thread block per head, the whole transform chain on chip.
//
// A real sequence of even length n is packed into a complex one of length N = n/2
// (odd n: length N = n with zero imaginary part). The complex transform is an in-place
// mixed-radix decimation-in-frequency FFT (radices 4, 2, 3, 5, 7 per thread, larger primes up
// to 127 as paired O(p^2) sums split over warps); its output is left in digit-reversed order and addressed through
// pos(k), and the inverse is the matching decimation-in-time chain, so no reordering pass
// and no second buffer is needed. Lengths with a larger prime factor go through a chirp-z
// (Bluestein) convolution of power-of-two length M >= 2N - 1 built from the same passes.
// The work buffer lives in shared memory when it fits, else in a per-block global scratch.
#include "common.cuh"
#include "select.cuh"

namespace akv {
namespace {

constexpr int kSssThreads = kSelThreads;  // 1024: select_topk runs in the same block

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
  return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 cmulc(float2 a, float2 b) {  // a * conj(b)
  return make_float2(fmaf(a.x, b.x, a.y * b.y), fmaf(a.y, b.x, -a.x * b.y));
}
__device__ __forceinline__ float2 cconj(float2 a) { return make_float2(a.x, -a.y); }
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cscale(float2 a, float s) { return make_float2(a.x * s, a.y * s); }
__device__ __forceinline__ float2 mul_i(float2 a) { return make_float2(-a.y, a.x); }    // i * a
__device__ __forceinline__ float2 mul_mi(float2 a) { return make_float2(a.y, -a.x); }   // -i * a

// cos / sin of 2 pi t / R for the odd radices handled per thread.
template <int R>
__device__ __forceinline__ float rcos(int t) {
  if (R == 3) return t == 0 ? 1.f : -0.5f;
  if (R == 5) return t == 0 ? 1.f : (t == 1 || t == 4) ? 0.30901699437494745f : -0.8090169943749475f;
  if (R == 7)
    return t == 0 ? 1.f
                  : (t == 1 || t == 6) ? 0.6234898018587336f
                                       : (t == 2 || t == 5) ? -0.2225209339563144f : -0.9009688679024191f;
  return 0.f;
}
template <int R>
__device__ __forceinline__ float rsin(int t) {
  if (R == 3) return t == 0 ? 0.f : t == 1 ? 0.8660254037844386f : -0.8660254037844386f;
  if (R == 5)
    return t == 0 ? 0.f
                  : t == 1 ? 0.9510565162951535f
                           : t == 2 ? 0.5877852522924731f : t == 3 ? -0.5877852522924731f : -0.9510565162951535f;
  if (R == 7)
    return t == 0 ? 0.f
                  : t == 1 ? 0.7818314824680298f
                           : t == 2 ? 0.9749279121818236f
                                    : t == 3 ? 0.4338837391175581f
                                             : t == 4 ? -0.4338837391175581f
                                                      : t == 5 ? -0.9749279121818236f : -0.7818314824680298f;
  return 0.f;
}

// In-register DFT of R points: X_c = sum_s v_s exp(-/+ 2 pi i s c / R)  (INV: plus sign).
template <int R, bool INV>
__device__ __forceinline__ void dft_small(float2* v) {
  if (R == 2) {
    float2 a = v[0], b = v[1];
    v[0] = cadd(a, b);
    v[1] = csub(a, b);
  } else if (R == 4) {
    float2 t0 = cadd(v[0], v[2]), t1 = csub(v[0], v[2]), t2 = cadd(v[1], v[3]), t3 = csub(v[1], v[3]);
    v[0] = cadd(t0, t2);
    v[2] = csub(t0, t2);
    float2 r = INV ? mul_i(t3) : mul_mi(t3);
    v[1] = cadd(t1, r);
    v[3] = csub(t1, r);
  } else {
    constexpr int H = (R - 1) / 2;
    float2 p[H + 1], q[H + 1];
#pragma unroll
    for (int s = 1; s <= H; ++s) {
      p[s] = cadd(v[s], v[R - s]);
      q[s] = csub(v[s], v[R - s]);
    }
    float2 v0 = v[0];
    float2 sum = v0;
#pragma unroll
    for (int s = 1; s <= H; ++s) sum = cadd(sum, p[s]);
    v[0] = sum;
#pragma unroll
    for (int c = 1; c <= H; ++c) {
      float2 A = v0, B = make_float2(0.f, 0.f);
#pragma unroll
      for (int s = 1; s <= H; ++s) {
        const float cc = rcos<R>((s * c) % R), ss = rsin<R>((s * c) % R);
        A.x = fmaf(p[s].x, cc, A.x);
        A.y = fmaf(p[s].y, cc, A.y);
        B.x = fmaf(q[s].x, ss, B.x);
        B.y = fmaf(q[s].y, ss, B.y);
      }
      // forward: X_c = A - i B, X_{R-c} = A + i B; inverse: the other way round
      float2 iB = mul_i(B);
      v[c] = INV ? cadd(A, iB) : csub(A, iB);
      v[R - c] = INV ? csub(A, iB) : cadd(A, iB);
    }
  }
}

// One in-place pass of radix R over sub-transforms of length ns (thread per butterfly).
// Forward (decimation in frequency): DFT_R, then multiply output c by W_ns^{j c}.
// Inverse (decimation in time): multiply input c by W_ns^{-j c}, then inverse DFT_R.
template <int R, bool INV>
__device__ __forceinline__ void pass_small(float2* buf, int N, int ns, const float2* __restrict__ tw) {
  const int m = ns / R, step = N / ns, nb = N / R;
  for (int t = threadIdx.x; t < nb; t += kSssThreads) {
    const int b = t / m, j = t - b * m;
    float2* p = buf + b * ns + j;
    float2 v[R];
#pragma unroll
    for (int s = 0; s < R; ++s) v[s] = p[s * m];
    if (!INV) {
      dft_small<R, false>(v);
      if (m > 1) {
#pragma unroll
        for (int c = 1; c < R; ++c) v[c] = cmul(v[c], __ldg(tw + j * c * step));
      }
    } else {
      if (m > 1) {
#pragma unroll
        for (int c = 1; c < R; ++c) v[c] = cmulc(v[c], __ldg(tw + j * c * step));
      }
      dft_small<R, true>(v);
    }
#pragma unroll
    for (int s = 0; s < R; ++s) p[s * m] = v[s];
  }
  __syncthreads();
}

// The same pass for an odd prime radix p, 11 <= p <= 127. A length-p DFT is O(p^2); pairing
// inputs s and p - s (P = a_s + a_{p-s}, Q = a_s - a_{p-s}) gives outputs c and p - c from the
// same real-by-complex products: X_c = A -/+ iB, A = a_0 + sum_s P_s cos(2 pi s c / p),
// B = sum_s Q_s sin(2 pi s c / p). Work is split into warp tasks: 32 consecutive butterflies
// (one per lane) times a chunk of kPrimeChunk output pairs, so the cos/sin reads are
// broadcasts. A round holds whole butterfly groups only: results stay in registers until
// every task of the round has read its inputs, then overwrite them.
constexpr int kPrimeChunk = 6;

template <bool INV>
__device__ __noinline__ void pass_prime(float2* buf, int N, int ns, int p, const float2* __restrict__ tw,
                                           float2* cs /* smem [128]: (cos, sin) of 2 pi t / p */) {
  __syncthreads();
  for (int t = threadIdx.x; t < p; t += kSssThreads) {
    const float2 w = __ldg(tw + t * (N / p));
    cs[t] = make_float2(w.x, -w.y);
  }
  __syncthreads();
  const int m = ns / p, step = N / ns, nb = N / p, H = (p - 1) / 2;
  const int n_chunks = (H + kPrimeChunk - 1) / kPrimeChunk;
  const int gpr = 32 / n_chunks;  // butterfly groups per round (n_chunks <= 11)
  const int n_groups = (nb + 31) / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = warp % n_chunks, c0 = 1 + chunk * kPrimeChunk;
  for (int g0 = 0; g0 < n_groups; g0 += gpr) {
    const int grp = g0 + warp / n_chunks;
    const int t = grp * 32 + lane;
    const bool active = warp < gpr * n_chunks && grp < n_groups && t < nb;
    float2 A[kPrimeChunk], B[kPrimeChunk];
    float2 X0 = make_float2(0.f, 0.f);
    float2* base = buf;
    int j = 0;
    if (active) {
      const int b = t / m;
      j = t - b * m;
      base = buf + b * ns + j;
      const float2 a0 = base[0];
      X0 = a0;
      int idx[kPrimeChunk];
#pragma unroll
      for (int o = 0; o < kPrimeChunk; ++o) {
        A[o] = a0;
        B[o] = make_float2(0.f, 0.f);
        idx[o] = c0 + o;  // (s * c) mod p at s = 1; c <= H + kPrimeChunk < p
        if (idx[o] >= p) idx[o] -= p;
      }
      for (int sI = 1; sI <= H; ++sI) {
        float2 x = base[sI * m], y = base[(p - sI) * m];
        if (INV && m > 1) {
          x = cmulc(x, __ldg(tw + j * sI * step));
          y = cmulc(y, __ldg(tw + j * (p - sI) * step));
        }
        const float2 P = cadd(x, y), Q = csub(x, y);
        X0 = cadd(X0, P);
#pragma unroll
        for (int o = 0; o < kPrimeChunk; ++o) {
          const float2 w = cs[idx[o]];
          A[o].x = fmaf(P.x, w.x, A[o].x);
          A[o].y = fmaf(P.y, w.x, A[o].y);
          B[o].x = fmaf(Q.x, w.y, B[o].x);
          B[o].y = fmaf(Q.y, w.y, B[o].y);
          idx[o] += c0 + o;
          if (idx[o] >= p) idx[o] -= p;  // c0 + o <= H + kPrimeChunk - 1 < p, so one step is enough
        }
      }
    }
    __syncthreads();
    if (active) {
      if (chunk == 0) base[0] = X0;
#pragma unroll
      for (int o = 0; o < kPrimeChunk; ++o) {
        const int c = c0 + o;
        if (c <= H) {
          const float2 iB = mul_i(B[o]);
          float2 xc = INV ? cadd(A[o], iB) : csub(A[o], iB);
          float2 xq = INV ? csub(A[o], iB) : cadd(A[o], iB);
          if (!INV && m > 1) {
            xc = cmul(xc, __ldg(tw + j * c * step));
            xq = cmul(xq, __ldg(tw + j * (p - c) * step));
          }
          base[c * m] = xc;
          base[(p - c) * m] = xq;
        }
      }
    }
    __syncthreads();
  }
}

template <bool INV>
__device__ __forceinline__ void one_pass(float2* buf, int N, int ns, int r, const float2* tw, float2* wp) {
  switch (r) {
    case 2: pass_small<2, INV>(buf, N, ns, tw); break;
    case 3: pass_small<3, INV>(buf, N, ns, tw); break;
    case 4: pass_small<4, INV>(buf, N, ns, tw); break;
    case 5: pass_small<5, INV>(buf, N, ns, tw); break;
    case 7: pass_small<7, INV>(buf, N, ns, tw); break;
    default: pass_prime<INV>(buf, N, ns, r, tw, wp); break;
  }
}

// Forward transform, natural order in, digit-reversed order out (see seq_pos).
__device__ __forceinline__ void fft_dif(float2* buf, const FftSeq& sq, const float2* tables, float2* wp) {
  const float2* tw = tables + sq.tw_offset;
  int ns = sq.N;
  for (int i = 0; i < sq.n_pass; ++i) {
    one_pass<false>(buf, sq.N, ns, sq.radix[i], tw, wp);
    ns /= sq.radix[i];
  }
}
// Inverse (unnormalised, sign +), digit-reversed order in, natural order out.
__device__ __forceinline__ void fft_dit_inv(float2* buf, const FftSeq& sq, const float2* tables, float2* wp) {
  const float2* tw = tables + sq.tw_offset;
  int ns = 1;
  for (int i = sq.n_pass - 1; i >= 0; --i) {
    ns *= sq.radix[i];
    one_pass<true>(buf, sq.N, ns, sq.radix[i], tw, wp);
  }
}
// Where the forward transform leaves bin k.
__device__ __forceinline__ int seq_pos(const FftSeq& sq, int k) {
  int len = sq.N, p = 0;
  for (int i = 0; i < sq.n_pass; ++i) {
    const int r = sq.radix[i];
    len /= r;
    const int q = k / r;
    p += (k - q * r) * len;
    k = q;
  }
  return p;
}

// Chirp-z: buf[0..N) holds y (natural order) on entry and DFT_N(y) (natural order) on exit.
// CONJ: conjugate on the way in and out, which turns the forward transform into the
// unnormalised inverse.
template <bool CONJ>
__device__ __forceinline__ void bluestein(float2* buf, const FftPlan& pl, const float2* tables, float2* wp) {
  const float2* chirp = tables + pl.chirp_offset;
  const float2* filt = tables + pl.filter_offset;
  const int N = pl.N, M = pl.M;
  for (int j = threadIdx.x; j < M; j += kSssThreads) {
    float2 v = make_float2(0.f, 0.f);
    if (j < N) {
      v = buf[j];
      if (CONJ) v = cconj(v);
      v = cmul(v, __ldg(chirp + j));
    }
    buf[j] = v;
  }
  __syncthreads();
  fft_dif(buf, pl.seq, tables, wp);
  for (int j = threadIdx.x; j < M; j += kSssThreads) buf[j] = cmul(buf[j], __ldg(filt + j));
  __syncthreads();
  fft_dit_inv(buf, pl.seq, tables, wp);
  for (int j = threadIdx.x; j < N; j += kSssThreads) {
    float2 v = cmul(buf[j], __ldg(chirp + j));
    buf[j] = CONJ ? cconj(v) : v;
  }
  __syncthreads();
}

__device__ __forceinline__ double block_sum(double v, double* red /* smem [32] */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  double t = red[lane];  // kSssThreads / 32 == 32 warps
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;
}

// Exclusive prefix of v over the block's threads (by thread index).
__device__ __forceinline__ double block_excl_scan(double v, double* red /* smem [32] */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) red[warp] = inc;
  __syncthreads();
  double wsum = red[lane];
  double winc = wsum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double t = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += t;
  }
  double wexcl = __shfl_sync(0xffffffffu, winc - wsum, warp);
  return wexcl + inc - v;
}

__global__ void __launch_bounds__(kSssThreads, 1)
sss_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const FftPlan* __restrict__ plans,
           const float2* __restrict__ tables, const float* scores, float* smoothed /* may alias scores */,
           int32_t* __restrict__ kstar_out, float2* __restrict__ scratch, int64_t scratch_per_block,
           const int32_t* __restrict__ budgets, const int32_t* __restrict__ cu_kept, int32_t* __restrict__ kept_idx,
           int* __restrict__ status) {
  extern __shared__ __align__(16) float2 sbuf[];
  __shared__ FftPlan pl;
  __shared__ float2 wp[128];
  __shared__ double red[32];
  __shared__ int s_kstar;
  __shared__ SelectSmem ssm;

  for (int u = blockIdx.x; u < sh.total_heads; u += gridDim.x) {
    const int r = u / sh.heads_per_req;
    const ReqDesc rq = reqs[r];
    __syncthreads();
    if (threadIdx.x == 0) {
      pl = plans[rq.fft_plan];
      s_kstar = 0x7fffffff;
    }
    __syncthreads();
    const int n = pl.n, N = pl.N, Kb = n / 2;
    float2* buf = pl.in_smem ? sbuf : scratch + static_cast<int64_t>(blockIdx.x) * scratch_per_block;
    const float* x = scores + rq.score_offset + static_cast<int64_t>(u - rq.head_base) * rq.P;
    float* y = smoothed ? smoothed + rq.score_offset + static_cast<int64_t>(u - rq.head_base) * rq.P : nullptr;

    // 1. load (packed: z_m = x_2m + i x_2m+1)
    if (pl.packed) {
      for (int m = threadIdx.x; m < N; m += kSssThreads) buf[m] = make_float2(x[2 * m], x[2 * m + 1]);
    } else {
      for (int m = threadIdx.x; m < N; m += kSssThreads) buf[m] = make_float2(x[m], 0.f);
    }
    __syncthreads();

    // 2. forward complex transform; bin k then sits at POS(k)
    if (pl.bluestein)
      bluestein<false>(buf, pl, tables, wp);
    else
      fft_dif(buf, pl.seq, tables, wp);
    const bool direct = !pl.bluestein;
    const int* pos_tab = reinterpret_cast<const int*>(tables + pl.pos_offset);  // where the forward pass left each bin
#define POS(k) (direct ? __ldg(pos_tab + (k)) : (k))

    // 3. packed: turn Z into the real sequence's spectrum F, pairwise in place.
    //    Slot of bin 0 holds (F_0, F_N), both real.
    const float2* post = tables + pl.post_offset;
    if (pl.packed) {
      for (int k = threadIdx.x; k <= N / 2; k += kSssThreads) {
        if (k == 0) {
          float2 z = buf[0];
          buf[0] = make_float2(z.x + z.y, z.x - z.y);
        } else if (2 * k == N) {
          const int pk = POS(k);
          buf[pk] = cconj(buf[pk]);
        } else {
          const int pk = POS(k), pq = POS(N - k);
          float2 zk = buf[pk], zq = cconj(buf[pq]);
          float2 E = cscale(cadd(zk, zq), 0.5f);
          float2 O = mul_mi(cscale(csub(zk, zq), 0.5f));
          float2 T = cmul(O, __ldg(post + k));
          buf[pk] = cadd(E, T);
          buf[pq] = cconj(csub(E, T));
        }
      }
      __syncthreads();
    }

    // 4. cumulative energy E(k) = sum_{i<=k} |F_i|^2 in fp64, and the smallest k with E(k) >= rho E(Kb)
    const int nbins = Kb + 1;
    const int per = (nbins + kSssThreads - 1) / kSssThreads;
    const int k0 = min(nbins, static_cast<int>(threadIdx.x) * per), k1 = min(nbins, k0 + per);
    auto energy = [&](int k) -> double {
      if (pl.packed) {
        if (k == 0) return static_cast<double>(buf[0].x) * buf[0].x;
        if (k == N) return static_cast<double>(buf[0].y) * buf[0].y;
      }
      float2 f = buf[POS(k)];
      return static_cast<double>(f.x) * f.x + static_cast<double>(f.y) * f.y;
    };
    double local = 0.0;
    for (int k = k0; k < k1; ++k) local += energy(k);
    const double before = block_excl_scan(local, red);
    const double total = block_sum(local, red);
    const double thr = static_cast<double>(sh.rho) * total;
    {
      double run = before;
      for (int k = k0; k < k1; ++k) {
        run += energy(k);
        if (run >= thr) {
          atomicMin(&s_kstar, k);
          break;
        }
      }
    }
    __syncthreads();
    const int kstar = min(s_kstar, Kb);
    if (threadIdx.x == 0 && kstar_out) kstar_out[u] = kstar;

    // 5. mask (1 up to k*, raised-cosine tail of T bins, 0 beyond) and the inverse of step 3
    const int T = sh.transition_bins;
    auto weight = [&](int k) -> float {
      if (k <= kstar) return 1.f;
      if (k <= kstar + T) return 0.5f * (1.f + cospif(static_cast<float>(k - kstar) / static_cast<float>(T + 1)));
      return 0.f;
    };
    if (pl.packed) {
      for (int k = threadIdx.x; k <= N / 2; k += kSssThreads) {
        if (k == 0) {
          float2 f = buf[0];
          const float f0 = f.x * weight(0), fN = f.y * weight(N);
          buf[0] = make_float2(0.5f * (f0 + fN), 0.5f * (f0 - fN));
        } else if (2 * k == N) {
          const int pk = POS(k);
          buf[pk] = cscale(cconj(buf[pk]), weight(k));
        } else {
          const int pk = POS(k), pq = POS(N - k);
          float2 fk = cscale(buf[pk], weight(k)), fq = cconj(cscale(buf[pq], weight(N - k)));
          float2 E = cscale(cadd(fk, fq), 0.5f);
          float2 Tt = cscale(csub(fk, fq), 0.5f);
          float2 O = cmulc(Tt, __ldg(post + k));
          float2 iO = mul_i(O);
          buf[pk] = cadd(E, iO);
          buf[pq] = cconj(csub(E, iO));
        }
      }
    } else {
      for (int k = threadIdx.x; k < N; k += kSssThreads) {
        const int kk = k <= Kb ? k : N - k;
        const int pk = POS(k);
        buf[pk] = cscale(buf[pk], weight(kk));
      }
    }
    __syncthreads();

    // 6. inverse complex transform (unnormalised), natural order out
    if (pl.bluestein)
      bluestein<true>(buf, pl, tables, wp);
    else
      fft_dit_inv(buf, pl.seq, tables, wp);
#undef POS

    // 7. residual mix. `smoothed` (optional) gets the result; when budgets are given the result
    //    also stays in the work buffer, as order-preserving keys, for the selection below.
    const float inv = 1.f / static_cast<float>(N), al = sh.alpha, om = 1.f - sh.alpha;
    const bool sel = budgets != nullptr;
    uint32_t* keys = reinterpret_cast<uint32_t*>(buf);
    if (pl.packed) {
      for (int m = threadIdx.x; m < N; m += kSssThreads) {
        float2 z = buf[m];
        const float x0 = x[2 * m], x1 = x[2 * m + 1];
        const float y0 = fmaf(al, z.x * inv, om * x0), y1 = fmaf(al, z.y * inv, om * x1);
        if (y) {
          y[2 * m] = y0;
          y[2 * m + 1] = y1;
        }
        if (sel) *reinterpret_cast<uint2*>(keys + 2 * m) = make_uint2(score_key(y0), score_key(y1));
      }
    } else {
      // key m lands in the slot of complex element m / 2: read a batch, then write it
      for (int m0 = 0; m0 < N; m0 += kSssThreads) {
        const int m = m0 + threadIdx.x;
        float ym = 0.f;
        if (m < N) {
          ym = fmaf(al, buf[m].x * inv, om * x[m]);
          if (y) y[m] = ym;
        }
        if (sel) {
          __syncthreads();
          if (m < N) keys[m] = score_key(ym);
          __syncthreads();
        }
      }
    }
    if (sel) {
      // 8. top-k of the smoothed scores, straight from the work buffer
      const int P = rq.P, W = sh.window;
      int k = budgets[u] - W;
      if (k < 0 || k > P) {
        if (threadIdx.x == 0) atomicExch(status, AUDIOKV_EDEVICE);
        k = k < 0 ? 0 : P;
      }
      __syncthreads();
      select_topk([&](int j) -> uint32_t { return keys[j]; }, P, W, k, kept_idx + cu_kept[u], &ssm, status);
    }
  }
}

// ---- tables ---------------------------------------------------------------------------
__global__ void fft_table_kernel(const FftPlan* __restrict__ plans, int n_plans, float2* __restrict__ tables) {
  const FftPlan pl = plans[blockIdx.y];
  const int gid = blockIdx.x * blockDim.x + threadIdx.x, gsz = gridDim.x * blockDim.x;
  const int Nt = pl.seq.N;
  for (int t = gid; t < Nt; t += gsz) {
    double s, c;
    sincospi(2.0 * t / Nt, &s, &c);
    tables[pl.seq.tw_offset + t] = make_float2(static_cast<float>(c), static_cast<float>(-s));
  }
  if (pl.packed) {
    for (int k = gid; k <= pl.N / 2; k += gsz) {
      double s, c;
      sincospi(2.0 * k / pl.n, &s, &c);
      tables[pl.post_offset + k] = make_float2(static_cast<float>(c), static_cast<float>(-s));
    }
  }
  if (!pl.bluestein) {
    int* pos_tab = reinterpret_cast<int*>(tables + pl.pos_offset);
    for (int k = gid; k < pl.N; k += gsz) pos_tab[k] = seq_pos(pl.seq, k);
  }
  if (pl.bluestein) {
    const int N = pl.N, M = pl.M;
    for (int j = gid; j < M; j += gsz) {
      // wrapped conjugate chirp b[j] = exp(+i pi j^2 / N) at j and M - j, j < N; zero elsewhere
      int jj = -1;
      if (j < N) jj = j;
      else if (M - j < N) jj = M - j;
      float2 b = make_float2(0.f, 0.f);
      if (jj >= 0) {
        const long long q = (static_cast<long long>(jj) * jj) % (2LL * N);
        double s, c;
        sincospi(static_cast<double>(q) / N, &s, &c);
        b = make_float2(static_cast<float>(c), static_cast<float>(s));
        if (j < N) tables[pl.chirp_offset + j] = make_float2(b.x, -b.y);
      }
      tables[pl.filter_offset + j] = b;
    }
  }
}

// Transforms each chirp-z filter in place (global memory) and folds in the 1/M of the inverse.
__global__ void __launch_bounds__(kSssThreads, 1)
fft_filter_kernel(const FftPlan* __restrict__ plans, float2* __restrict__ tables) {
  __shared__ FftPlan pl;
  __shared__ float2 wp[128];
  if (threadIdx.x == 0) pl = plans[blockIdx.x];
  __syncthreads();
  if (!pl.bluestein) return;
  float2* f = tables + pl.filter_offset;
  fft_dif(f, pl.seq, tables, wp);
  const float inv = 1.f / static_cast<float>(pl.M);
  for (int j = threadIdx.x; j < pl.M; j += kSssThreads) f[j] = cscale(f[j], inv);
}

}  // namespace

cudaError_t launch_fft_tables(int n_plans, float2* d_tables, const FftPlan* d_plans, Launch ln) {
  fft_table_kernel<<<dim3(32, n_plans), 256, 0, ln.stream>>>(d_plans, n_plans, d_tables);
  ln.done("fft_table");
  fft_filter_kernel<<<n_plans, kSssThreads, 0, ln.stream>>>(d_plans, d_tables);
  ln.done("fft_filter");
  return cudaGetLastError();
}

cudaError_t launch_sss(const Shape& sh, const ReqDesc* d_reqs, const FftPlan* d_plans, const float2* d_tables,
                       const float* scores, float* smoothed, int32_t* kstar, float2* scratch,
                       int64_t scratch_per_block, int grid, size_t smem_bytes, const int32_t* budgets,
                       const int32_t* cu_kept, int32_t* kept_idx, int* status, Launch ln) {
  cudaError_t e = cudaFuncSetAttribute(sss_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  sss_kernel<<<grid, kSssThreads, smem_bytes, ln.stream>>>(sh, d_reqs, d_plans, d_tables, scores, smoothed, kstar,
                                                           scratch, scratch_per_block, budgets, cu_kept, kept_idx,
                                                           status);
  ln.done(budgets ? "sss_select" : "sss");
  return cudaGetLastError();
}

}  // namespace akv
