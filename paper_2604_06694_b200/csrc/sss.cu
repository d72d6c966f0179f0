// Spectral Score Smoothing: one thread block per head, the whole transform chain on chip.
//
// A real sequence of even length n is packed into a complex one of length N = n/2
// (odd n: length N = n with zero imaginary part). The complex transform is an in-place
// mixed-radix decimation-in-frequency FFT (radices 2 to 19 one butterfly per thread, larger primes up
// to 127 as paired O(p^2) sums, one output pair of one butterfly per task); its output is left in digit-reversed order and addressed through
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

// The work buffer of a transform. In shared memory element i lives at i + (i >> 4): the passes of an in-place
// transform read with power-of-two strides (and the late ones with strides of a few elements between
// neighbouring threads), which without the skew puts many lanes on the same banks. sh = 31 switches the skew
// off (global scratch, tables).
struct SkewBuf {
  float2* p;
  int sh;
  int off;
  __device__ __forceinline__ float2& operator[](int i) const {
    const int e = off + i;
    return p[e + (e >> sh)];
  }
  __device__ __forceinline__ SkewBuf operator+(int d) const { return SkewBuf{p, sh, off + d}; }
};

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
__device__ __forceinline__ void pass_small(SkewBuf buf, int N, int ns, const float2* tw) {
  const int m = ns / R, step = N / ns, nb = N / R;
  for (int t = threadIdx.x; t < nb; t += kSssThreads) {
    const int b = t / m, j = t - b * m;
    const SkewBuf p = buf + (b * ns + j);
    float2 v[R];
#pragma unroll
    for (int s = 0; s < R; ++s) v[s] = p[s * m];
    if (!INV) {
      dft_small<R, false>(v);
      if (m > 1) {
#pragma unroll
        for (int c = 1; c < R; ++c) v[c] = cmul(v[c], tw[j * c * step]);
      }
    } else {
      if (m > 1) {
#pragma unroll
        for (int c = 1; c < R; ++c) v[c] = cmulc(v[c], tw[j * c * step]);
      }
      dft_small<R, true>(v);
    }
#pragma unroll
    for (int s = 0; s < R; ++s) p[s * m] = v[s];
  }
  __syncthreads();
}

// cos / sin of 2 pi t / R for the odd radices handled by one thread per butterfly with streamed outputs.
template <int R>
__device__ __forceinline__ float ocos(int t) {
  if (R == 11) {
    switch (t) {
      case 0: return 1.0f;
      case 1: return 0.84125353283118121f;
      case 2: return 0.41541501300188644f;
      case 3: return -0.142314838273285f;
      case 4: return -0.65486073394528499f;
      case 5: return -0.95949297361449737f;
      case 6: return -0.95949297361449748f;
      case 7: return -0.65486073394528521f;
      case 8: return -0.14231483827328523f;
      case 9: return 0.41541501300188605f;
      case 10: return 0.84125353283118121f;
    }
  }
  if (R == 13) {
    switch (t) {
      case 0: return 1.0f;
      case 1: return 0.88545602565320991f;
      case 2: return 0.56806474673115592f;
      case 3: return 0.12053668025532301f;
      case 4: return -0.35460488704253545f;
      case 5: return -0.74851074817110119f;
      case 6: return -0.97094181742605201f;
      case 7: return -0.97094181742605212f;
      case 8: return -0.7485107481711013f;
      case 9: return -0.3546048870425359f;
      case 10: return 0.1205366802553232f;
      case 11: return 0.56806474673115481f;
      case 12: return 0.88545602565321002f;
    }
  }
  if (R == 17) {
    switch (t) {
      case 0: return 1.0f;
      case 1: return 0.93247222940435581f;
      case 2: return 0.73900891722065909f;
      case 3: return 0.44573835577653831f;
      case 4: return 0.092268359463302016f;
      case 5: return -0.27366299007208289f;
      case 6: return -0.60263463637925629f;
      case 7: return -0.85021713572961399f;
      case 8: return -0.98297309968390179f;
      case 9: return -0.98297309968390179f;
      case 10: return -0.8502171357296141f;
      case 11: return -0.60263463637925718f;
      case 12: return -0.27366299007208311f;
      case 13: return 0.092268359463302432f;
      case 14: return 0.4457383557765377f;
      case 15: return 0.73900891722065853f;
      case 16: return 0.93247222940435581f;
    }
  }
  if (R == 19) {
    switch (t) {
      case 0: return 1.0f;
      case 1: return 0.94581724170063464f;
      case 2: return 0.78914050939639357f;
      case 3: return 0.54694815812242692f;
      case 4: return 0.24548548714079924f;
      case 5: return -0.082579345472332269f;
      case 6: return -0.40169542465296942f;
      case 7: return -0.67728157162574087f;
      case 8: return -0.87947375120648896f;
      case 9: return -0.98636130340272232f;
      case 10: return -0.98636130340272243f;
      case 11: return -0.8794737512064893f;
      case 12: return -0.6772815716257411f;
      case 13: return -0.40169542465296904f;
      case 14: return -0.082579345472332741f;
      case 15: return 0.24548548714079879f;
      case 16: return 0.54694815812242659f;
      case 17: return 0.78914050939639391f;
      case 18: return 0.94581724170063464f;
    }
  }
  return 0.f;
}
template <int R>
__device__ __forceinline__ float osin(int t) {
  if (R == 11) {
    switch (t) {
      case 0: return 0.0f;
      case 1: return 0.54064081745559756f;
      case 2: return 0.90963199535451833f;
      case 3: return 0.9898214418809328f;
      case 4: return 0.75574957435425827f;
      case 5: return 0.28173255684142967f;
      case 6: return -0.28173255684142939f;
      case 7: return -0.75574957435425816f;
      case 8: return -0.98982144188093268f;
      case 9: return -0.90963199535451855f;
      case 10: return -0.54064081745559744f;
    }
  }
  if (R == 13) {
    switch (t) {
      case 0: return 0.0f;
      case 1: return 0.46472317204376851f;
      case 2: return 0.82298386589365635f;
      case 3: return 0.99270887409805397f;
      case 4: return 0.93501624268541483f;
      case 5: return 0.66312265824079519f;
      case 6: return 0.23931566428755768f;
      case 7: return -0.23931566428755743f;
      case 8: return -0.66312265824079497f;
      case 9: return -0.93501624268541472f;
      case 10: return -0.99270887409805397f;
      case 11: return -0.82298386589365702f;
      case 12: return -0.4647231720437684f;
    }
  }
  if (R == 17) {
    switch (t) {
      case 0: return 0.0f;
      case 1: return 0.36124166618715292f;
      case 2: return 0.67369564364655721f;
      case 3: return 0.89516329135506234f;
      case 4: return 0.99573417629503447f;
      case 5: return 0.96182564317281904f;
      case 6: return 0.7980172272802396f;
      case 7: return 0.52643216287735606f;
      case 8: return 0.18374951781657037f;
      case 9: return -0.18374951781657012f;
      case 10: return -0.52643216287735584f;
      case 11: return -0.79801722728023894f;
      case 12: return -0.96182564317281904f;
      case 13: return -0.99573417629503447f;
      case 14: return -0.89516329135506256f;
      case 15: return -0.67369564364655776f;
      case 16: return -0.36124166618715303f;
    }
  }
  if (R == 19) {
    switch (t) {
      case 0: return 0.0f;
      case 1: return 0.32469946920468346f;
      case 2: return 0.61421271268966782f;
      case 3: return 0.83716647826252855f;
      case 4: return 0.96940026593933037f;
      case 5: return 0.99658449300666985f;
      case 6: return 0.9157733266550574f;
      case 7: return 0.73572391067313181f;
      case 8: return 0.47594739303707367f;
      case 9: return 0.16459459028073403f;
      case 10: return -0.16459459028073378f;
      case 11: return -0.47594739303707312f;
      case 12: return -0.73572391067313159f;
      case 13: return -0.91577332665505762f;
      case 14: return -0.99658449300666985f;
      case 15: return -0.96940026593933049f;
      case 16: return -0.83716647826252877f;
      case 17: return -0.61421271268966737f;
      case 18: return -0.32469946920468373f;
    }
  }
  return 0.f;
}

// One in-place pass of an odd radix R in {11, 13, 17, 19}: one thread per butterfly. The inputs are folded into
// P_s = a_s + a_{R-s}, Q_s = a_s - a_{R-s} (kept in registers); outputs c and R - c come from the same
// real-by-complex products, X_c = A -/+ iB with A = a_0 + sum_s P_s cos(2 pi s c / R), B = sum_s Q_s sin(2 pi s c / R),
// and are written back as soon as they are complete.
template <int R, bool INV>
__device__ __noinline__ void pass_odd(SkewBuf buf, int N, int ns, const float2* tw) {
  constexpr int H = (R - 1) / 2;
  const int m = ns / R, step = N / ns, nb = N / R;
  for (int t = threadIdx.x; t < nb; t += kSssThreads) {
    const int b = t / m, j = t - b * m;
    const SkewBuf p = buf + (b * ns + j);
    const float2 v0 = p[0];
    float2 P[H], Q[H];
    float2 sum = v0;
#pragma unroll
    for (int sI = 1; sI <= H; ++sI) {
      float2 x = p[sI * m], y = p[(R - sI) * m];
      if (INV && m > 1) {
        x = cmulc(x, tw[j * sI * step]);
        y = cmulc(y, tw[j * (R - sI) * step]);
      }
      P[sI - 1] = cadd(x, y);
      Q[sI - 1] = csub(x, y);
      sum = cadd(sum, P[sI - 1]);
    }
    p[0] = sum;
#pragma unroll
    for (int c = 1; c <= H; ++c) {
      float2 A = v0, B = make_float2(0.f, 0.f);
#pragma unroll
      for (int sI = 1; sI <= H; ++sI) {
        const float cc = ocos<R>((sI * c) % R), ss = osin<R>((sI * c) % R);
        A.x = fmaf(P[sI - 1].x, cc, A.x);
        A.y = fmaf(P[sI - 1].y, cc, A.y);
        B.x = fmaf(Q[sI - 1].x, ss, B.x);
        B.y = fmaf(Q[sI - 1].y, ss, B.y);
      }
      const float2 iB = mul_i(B);
      float2 xc = INV ? cadd(A, iB) : csub(A, iB);
      float2 xq = INV ? csub(A, iB) : cadd(A, iB);
      if (!INV && m > 1) {
        xc = cmul(xc, tw[j * c * step]);
        xq = cmul(xq, tw[j * (R - c) * step]);
      }
      p[c * m] = xc;
      p[(R - c) * m] = xq;
    }
  }
  __syncthreads();
}

// The same pass for an odd prime radix p, 23 <= p <= 127 (11 to 19 have pass_odd). A length-p DFT is O(p^2); pairing
// inputs s and p - s (P = a_s + a_{p-s}, Q = a_s - a_{p-s}) gives outputs c and p - c from the
// same real-by-complex products: X_c = A -/+ iB, A = a_0 + sum_s P_s cos(2 pi s c / p),
// B = sum_s Q_s sin(2 pi s c / p); c = 0 is the plain sum. One task = one butterfly and kPrimeOut
// consecutive c in [0, (p-1)/2]; consecutive threads take consecutive butterflies of the same c, so
// the data reads are contiguous and the cos/sin reads are broadcasts. A thread keeps the results of
// its (at most kPrimeTasks) tasks in registers until every task of the round has read its inputs.
// The pass twiddles are applied in a sweep of their own (inverse: before, forward: with the
// write-back).
constexpr int kPrimeTasks = 1;  // tasks per thread and round (two were tried: the second slot is mostly empty and costs registers)
constexpr int kPrimeOut = 5;    // consecutive c per task: the folded inputs P_s, Q_s are formed once for all of them

template <bool INV>
__device__ __noinline__ void pass_prime(SkewBuf buf, int N, int ns, int p, const float2* tw,
                                        float2* cs /* smem [128]: (cos, sin) of 2 pi t / p */) {
  __syncthreads();
  for (int t = threadIdx.x; t < p; t += kSssThreads) {
    const float2 w = tw[t * (N / p)];
    cs[t] = make_float2(w.x, -w.y);
  }
  const int m = ns / p, step = N / ns, nb = N / p, H = (p - 1) / 2;
  if (INV && m > 1) {
    // element e = b ns + s m + j gets W_ns^{-j s}
    for (int e = threadIdx.x; e < N; e += kSssThreads) {
      const int r = e % ns, sI = r / m, j = r - sI * m;
      if (sI > 0 && j > 0) buf[e] = cmulc(buf[e], tw[j * sI * step]);
    }
  }
  __syncthreads();
  const int n_chunks = (H + kPrimeOut) / kPrimeOut;  // chunks of c over [0, H]
  const int per_round = max(1, (kPrimeTasks * kSssThreads) / n_chunks);  // butterflies per round
  for (int b0 = 0; b0 < nb; b0 += per_round) {
    const int nbr = min(per_round, nb - b0);
    const int n_task = nbr * n_chunks;
    float2 A[kPrimeTasks][kPrimeOut], B[kPrimeTasks][kPrimeOut];
#pragma unroll
    for (int i = 0; i < kPrimeTasks; ++i) {
      const int q = threadIdx.x + kSssThreads * i;
#pragma unroll
      for (int o = 0; o < kPrimeOut; ++o) A[i][o] = B[i][o] = make_float2(0.f, 0.f);
      if (q < n_task) {
        const int chunk = q / nbr;
        const int t = b0 + q - chunk * nbr;
        const int b = t / m, j = t - b * m;
        const SkewBuf base = buf + (b * ns + j);
        const float2 a0 = base[0];
        int idx[kPrimeOut];
#pragma unroll
        for (int o = 0; o < kPrimeOut; ++o) {
          A[i][o] = a0;
          idx[o] = chunk * kPrimeOut + o;  // (s c) mod p at s = 1; c <= H + kPrimeOut - 1 < p
        }
        for (int sI = 1; sI <= H; ++sI) {
          const float2 x = base[sI * m], y = base[(p - sI) * m];
          const float2 P = cadd(x, y), Q = csub(x, y);
#pragma unroll
          for (int o = 0; o < kPrimeOut; ++o) {
            const float2 w = cs[idx[o]];
            A[i][o].x = fmaf(P.x, w.x, A[i][o].x);
            A[i][o].y = fmaf(P.y, w.x, A[i][o].y);
            B[i][o].x = fmaf(Q.x, w.y, B[i][o].x);
            B[i][o].y = fmaf(Q.y, w.y, B[i][o].y);
            idx[o] += chunk * kPrimeOut + o;
            if (idx[o] >= p) idx[o] -= p;
          }
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kPrimeTasks; ++i) {
      const int q = threadIdx.x + kSssThreads * i;
      if (q < n_task) {
        const int chunk = q / nbr;
        const int t = b0 + q - chunk * nbr;
        const int b = t / m, j = t - b * m;
        const SkewBuf base = buf + (b * ns + j);
#pragma unroll
        for (int o = 0; o < kPrimeOut; ++o) {
          const int c = chunk * kPrimeOut + o;
          if (c == 0) {
            base[0] = A[i][o];
          } else if (c <= H) {
            const float2 iB = mul_i(B[i][o]);
            float2 xc = INV ? cadd(A[i][o], iB) : csub(A[i][o], iB);
            float2 xq = INV ? csub(A[i][o], iB) : cadd(A[i][o], iB);
            if (!INV && m > 1) {
              xc = cmul(xc, tw[j * c * step]);
              xq = cmul(xq, tw[j * (p - c) * step]);
            }
            base[c * m] = xc;
            base[(p - c) * m] = xq;
          }
        }
      }
    }
    __syncthreads();
  }
}

template <bool INV>
__device__ __forceinline__ void one_pass(SkewBuf buf, int N, int ns, int r, const float2* tw, float2* wp) {
  switch (r) {
    case 2: pass_small<2, INV>(buf, N, ns, tw); break;
    case 3: pass_small<3, INV>(buf, N, ns, tw); break;
    case 4: pass_small<4, INV>(buf, N, ns, tw); break;
    case 5: pass_small<5, INV>(buf, N, ns, tw); break;
    case 7: pass_small<7, INV>(buf, N, ns, tw); break;
    case 11: pass_odd<11, INV>(buf, N, ns, tw); break;
    case 13: pass_odd<13, INV>(buf, N, ns, tw); break;
    case 17: pass_odd<17, INV>(buf, N, ns, tw); break;
    case 19: pass_odd<19, INV>(buf, N, ns, tw); break;
    default: pass_prime<INV>(buf, N, ns, r, tw, wp); break;
  }
}

// Forward transform, natural order in, digit-reversed order out (see seq_pos).
// tw: W_N^t = exp(-2 pi i t / N), t in [0, N); in shared or global memory.
__device__ __noinline__ void fft_dif(SkewBuf buf, const FftSeq& sq, const float2* tw, float2* wp) {
  int ns = sq.N;
  for (int i = 0; i < sq.n_pass; ++i) {
    one_pass<false>(buf, sq.N, ns, sq.radix[i], tw, wp);
    ns /= sq.radix[i];
  }
}
// Inverse (unnormalised, sign +), digit-reversed order in, natural order out.
__device__ __noinline__ void fft_dit_inv(SkewBuf buf, const FftSeq& sq, const float2* tw, float2* wp) {
  int ns = 1;
  for (int i = sq.n_pass - 1; i >= 0; --i) {
    ns *= sq.radix[i];
    one_pass<true>(buf, sq.N, ns, sq.radix[i], tw, wp);
  }
}
// The same two transforms for a buffer in global memory that is too long for shared memory. The first g passes
// of the forward transform couple elements that lie far apart and run on the global buffer; after them the
// transform falls apart into F = r_1 ... r_g contiguous blocks of length len = N / F, each of which is brought
// into shared memory (with its own twiddles W_len^t = W_N^{t F}) for the remaining passes. The inverse runs the
// steps backwards. Every element then makes g + 1 round trips to global memory instead of one per pass.
__device__ __noinline__ void fft_dif_big(SkewBuf gbuf, const FftSeq& sq, int g, const float2* tw, float2* wp,
                                         float2* sbuf) {
  int ns = sq.N;
  for (int i = 0; i < g; ++i) {
    one_pass<false>(gbuf, sq.N, ns, sq.radix[i], tw, wp);
    ns /= sq.radix[i];
  }
  const int len = ns, F = sq.N / len;
  const SkewBuf sb{sbuf, 4, 0};
  float2* s_tw = sbuf + sss_padded(len);
  __syncthreads();
  for (int t = threadIdx.x; t < len; t += kSssThreads) s_tw[t] = tw[t * F];
  for (int blk = 0; blk < F; ++blk) {
    __syncthreads();
    for (int t = threadIdx.x; t < len; t += kSssThreads) sb[t] = gbuf[blk * len + t];
    __syncthreads();
    int ns2 = len;
    for (int i = g; i < sq.n_pass; ++i) {
      one_pass<false>(sb, len, ns2, sq.radix[i], s_tw, wp);
      ns2 /= sq.radix[i];
    }
    for (int t = threadIdx.x; t < len; t += kSssThreads) gbuf[blk * len + t] = sb[t];
  }
  __syncthreads();
}
__device__ __noinline__ void fft_dit_inv_big(SkewBuf gbuf, const FftSeq& sq, int g, const float2* tw, float2* wp,
                                             float2* sbuf) {
  int len = sq.N;
  for (int i = 0; i < g; ++i) len /= sq.radix[i];
  const int F = sq.N / len;
  const SkewBuf sb{sbuf, 4, 0};
  float2* s_tw = sbuf + sss_padded(len);
  __syncthreads();
  for (int t = threadIdx.x; t < len; t += kSssThreads) s_tw[t] = tw[t * F];
  for (int blk = 0; blk < F; ++blk) {
    __syncthreads();
    for (int t = threadIdx.x; t < len; t += kSssThreads) sb[t] = gbuf[blk * len + t];
    __syncthreads();
    int ns2 = 1;
    for (int i = sq.n_pass - 1; i >= g; --i) {
      ns2 *= sq.radix[i];
      one_pass<true>(sb, len, ns2, sq.radix[i], s_tw, wp);
    }
    for (int t = threadIdx.x; t < len; t += kSssThreads) gbuf[blk * len + t] = sb[t];
  }
  __syncthreads();
  int ns = len;
  for (int i = g - 1; i >= 0; --i) {
    ns *= sq.radix[i];
    one_pass<true>(gbuf, sq.N, ns, sq.radix[i], tw, wp);
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

// Chirp-z: buf[0..n_in) holds y (natural order; entries from n_in on count as zero) on entry and bins 0..n_out-1
// of DFT_N(y) (natural order) on exit. `filt` is the transformed wrapped chirp that fits this pair of ranges: the
// plan's filter for n_in = n_out = N, and for a half plan the filter (N in, (N+1)/2 out) or filter2 ((N+1)/2 in,
// N out). CONJ: conjugate on the way in and out, which turns the forward transform into the unnormalised inverse.
template <bool CONJ>
__device__ __forceinline__ void bluestein(SkewBuf buf, const FftPlan& pl, const float2* tables, float2* wp, float2* sbuf,
                                          int n_in, int n_out, const float2* filt) {
  const float2* chirp = tables + pl.chirp_offset;
  const int M = pl.M;
  for (int j = threadIdx.x; j < M; j += kSssThreads) {
    float2 v = make_float2(0.f, 0.f);
    if (j < n_in) {
      v = buf[j];
      if (CONJ) v = cconj(v);
      v = cmul(v, __ldg(chirp + j));
    }
    buf[j] = v;
  }
  __syncthreads();
  if (pl.in_smem) fft_dif(buf, pl.seq, tables + pl.seq.tw_offset, wp);
  else fft_dif_big(buf, pl.seq, pl.g_pass, tables + pl.seq.tw_offset, wp, sbuf);
  for (int j = threadIdx.x; j < M; j += kSssThreads) buf[j] = cmul(buf[j], __ldg(filt + j));
  __syncthreads();
  if (pl.in_smem) fft_dit_inv(buf, pl.seq, tables + pl.seq.tw_offset, wp);
  else fft_dit_inv_big(buf, pl.seq, pl.g_pass, tables + pl.seq.tw_offset, wp, sbuf);
  for (int j = threadIdx.x; j < n_out; j += kSssThreads) {
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

// ---- low cut-offs without a transform ---------------------------------------------------------------------------
// Attention scores are positive, so their mean usually carries most of the energy and k* is a handful of bins. The
// block then evaluates those bins directly, O(n (k* + T)) operations instead of two transforms of n points: the
// total energy comes from Parseval's identity (sum of squares in fp64), the first kDirectBins bins from their
// definition. The shortcut is taken only when those bins decide k* with a clear margin and k* + T lies inside them;
// otherwise the transform path decides.
constexpr int kDirectBins = 12;
constexpr int kDirectRows = 64;  // entries per thread the table covers: even n up to 131072, odd n up to 65535
constexpr int kDirectRegs = 8;   // entries per thread held in registers

// Entry m = t + kSssThreads i of thread t holds token m (odd n) or tokens 2m and 2m + 1 (even n): token j = a m + b.
// With w_k = e^{-2 pi i k / n},  w_k^j = w_k^{a t} * w_k^b * w_k^{a kSssThreads i}: the first factor is a power of one
// rotation per thread, the second a power of one rotation per head, the third comes from a table of
// rows x kDirectBins entries built once per head. A bin then costs one shared-memory read and two FMAs per token.
// The code is kept short on purpose: it runs once per head and launch, mostly from a cold instruction cache; for the
// same reason it is inlined into the kernel, next to the code that runs before and after it (out of line the
// benchmark's smoothing kernel took 29.2 instead of 28.1 us, at L = 32768 62.5 instead of 58.0).
struct DirectSmem {
  float2 tab[kDirectRows][kDirectBins];          // tab[i][k] = w_k^{a kSssThreads i}
  float2 part[kSssThreads / 32][kDirectBins];    // per warp: bins 1 .. kDirectBins - 1
  double sums[kSssThreads / 32][3];              // per warp: sum x, sum x^2, alternating sum
  double energy[kDirectBins];                    // |F_k|^2 as it counts towards the cumulative energy
  double tot[3];                                 // F_0 (= sum x), the energy threshold rho E, the margin of a decision
  float2 bin[kDirectBins];                       // F_k
  int kstar;                                     // stage 1: k*, -1: left to the transform, -2: the bins decide
  int k_hi;                                      // last bin to evaluate; after stage 3: k* or -1
};

// e^{-2 pi i (j k mod n) / n}: the product is reduced exactly in integers, the angle then lies in [-pi, pi] where the
// fast sine and cosine are good to 5e-7.
__device__ __forceinline__ float2 unit_root(int j, int k, int n, float inv_n, float two_pi_over_n) {
  const int jk = j * k;                                   // j <= 2^17, k < 16
  int m = jk - n * __float2int_rd(static_cast<float>(jk) * inv_n);
  m += m < 0 ? n : 0;
  m -= m >= n ? n : 0;
  m -= 2 * m > n ? n : 0;                                 // (-n/2, n/2]
  float sn, cs;
  __sincosf(static_cast<float>(m) * two_pi_over_n, &sn, &cs);
  return make_float2(cs, -sn);
}

// e^{-2 pi i j / n} for 0 <= j < 2^22, to fp32 rounding
__device__ __forceinline__ float2 unit_root_exact(int j, int n) {
  int m = j % n;
  m -= 2 * m > n ? n : 0;  // (-n/2, n/2]: the quotient below is rounded relative to an angle of at most pi
  float sn, cs;
  sincospif(static_cast<float>(2 * m) / static_cast<float>(n), &sn, &cs);
  return make_float2(cs, -sn);
}

struct DirectGeom {
  int a, M, rows;          // tokens per entry, entries, entries per thread
  float2 wt, v;            // w_1^{a t}, w_1
};

__device__ __forceinline__ DirectGeom direct_geom(int n, bool packed) {
  DirectGeom g;
  g.a = packed ? 2 : 1;
  g.M = n / g.a;
  g.rows = (g.M + kSssThreads - 1) / kSssThreads;
  // one accurate rotation per thread, w_1^t; w_1 is the ratio of two neighbours' and w_1^{2t} its square
  const float2 w = unit_root_exact(threadIdx.x, n);
  const float2 w_l0 = make_float2(__shfl_sync(0xffffffffu, w.x, 0), __shfl_sync(0xffffffffu, w.y, 0));
  const float2 w_l1 = make_float2(__shfl_sync(0xffffffffu, w.x, 1), __shfl_sync(0xffffffffu, w.y, 1));
  g.v = cmulc(w_l1, w_l0);
  g.wt = packed ? cmul(w, w) : w;
  return g;
}

// x: the n scores of the head (rows <= kDirectRows); T: bins of the cosine band. Returns k* (and leaves the bins in
// ds->bin and the table in ds->tab) or -1 when the transform has to decide.
__device__ __forceinline__ int direct_cutoff(const float* __restrict__ x, int n, bool packed, const DirectGeom& g, int smooth_mode,
                                         float rho, float kappa, int T, DirectSmem* ds) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();  // ds may still be read by the head before
  {
    const float inv_n = 1.f / static_cast<float>(n), tpn = 6.283185307179586f * inv_n;
    for (int e = threadIdx.x; e < g.rows * kDirectBins; e += kSssThreads) {
      const int i = e / kDirectBins, k = e - i * kDirectBins;
      ds->tab[i][k] = unit_root(g.a * kSssThreads * i, k, n, inv_n, tpn);
    }
  }
  // the thread's first entries stay in registers; the plain, squared and alternating sums are kept in fp64
  float x0[kDirectRegs], x1[kDirectRegs];
  double sx = 0.0, sxx = 0.0, salt = 0.0;
#pragma unroll
  for (int i = 0; i < kDirectRegs; ++i) {
    const int m = threadIdx.x + kSssThreads * i;
    x0[i] = m < g.M ? x[g.a * m] : 0.f;
    x1[i] = (packed && m < g.M) ? x[g.a * m + 1] : 0.f;
  }
  const bool even_entry = packed || (threadIdx.x & 1) == 0;  // kSssThreads is even: all of a thread's tokens m alike
#pragma unroll
  for (int i = 0; i < kDirectRegs; ++i) {
    const double d0 = static_cast<double>(x0[i]), d1 = static_cast<double>(x1[i]);
    sx += d0 + d1;
    sxx = fma(d0, d0, fma(d1, d1, sxx));
    salt += even_entry ? d0 - d1 : -d0;
  }
  for (int i = kDirectRegs; i < g.rows; ++i) {
    const int m = threadIdx.x + kSssThreads * i;
    if (m >= g.M) break;
    const double d0 = static_cast<double>(x[g.a * m]), d1 = packed ? static_cast<double>(x[g.a * m + 1]) : 0.0;
    sx += d0 + d1;
    sxx = fma(d0, d0, fma(d1, d1, sxx));
    salt += even_entry ? d0 - d1 : -d0;
  }
#pragma unroll 1
  for (int q = 0; q < 3; ++q) {
    double val = q == 0 ? sx : (q == 1 ? sxx : salt);
    for (int o = 16; o > 0; o >>= 1) val += __shfl_xor_sync(0xffffffffu, val, o);
    if (lane == 0) ds->sums[warp][q] = val;
  }
  __syncthreads();  // the table and the warps' sums are complete
  // Stage 1, from the three sums alone (warp 0): the mean bin F_0 and, by Parseval, the total over the bins
  // 0 .. floor(n/2). Often that settles the cut-off at bin 0, and only the T bins of the cosine band are needed; it
  // also tells a head whose mean holds less than half of the energy asked for, which is left to the transform at once
  // (a matter of time only: both paths compute the same function).
  if (warp == 0) {
    double t[3];
#pragma unroll 1
    for (int q = 0; q < 3; ++q) {
      double v = ds->sums[lane][q];
#pragma unroll 1
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      t[q] = v;
    }
    if (lane == 0) {
      const int Kb = n / 2;
      const double F0 = t[0], FN = t[2];
      const double total = 0.5 * (static_cast<double>(n) * t[1] + F0 * F0 + ((n & 1) ? 0.0 : FN * FN));
      const bool no_mean = smooth_mode == AUDIOKV_SMOOTH_ENERGY_NO_MEAN;
      const double rest = fmax(total - F0 * F0, 0.0), whole = no_mean ? rest : total;
      const double thr = static_cast<double>(rho) * whole;
      // The rotations are good to about 1e-6, so a bin's energy is off by up to 2e-6 |F_k| F_0: a decision is taken
      // here only when it is clear of the threshold by several times the sum of that over the bins.
      const double margin = 1e-5 * (whole + fabs(F0) * static_cast<double>(sqrtf(static_cast<float>(rest))));
      int ks = -2, k_hi = kDirectBins - 1;  // -2: the bins have to decide
      if (smooth_mode == AUDIOKV_SMOOTH_FIXED_FRACTION) {
        ks = static_cast<int>(floor(static_cast<double>(kappa) * Kb));
      } else if (!(whole > 0.0)) {
        ks = -1;
      } else if (!no_mean) {
        if (F0 * F0 >= thr + margin) ks = 0;
        else if (F0 * F0 < 0.5 * thr) ks = -1;
      }
      if (ks >= 0) {
        k_hi = ks + T;
        if (k_hi >= kDirectBins || k_hi >= Kb) ks = -1;
      }
      ds->tot[0] = F0;
      ds->tot[1] = thr;
      ds->tot[2] = margin;
      ds->bin[0] = make_float2(static_cast<float>(F0), 0.f);
      ds->energy[0] = no_mean ? 0.0 : F0 * F0;
      ds->k_hi = k_hi;
      ds->kstar = ks;
    }
  }
  __syncthreads();
  if (ds->kstar == -1) return -1;
  const int k_hi = ds->k_hi;
  // Stage 2: bins 1 .. k_hi from their definition
  float2 pk = make_float2(1.f, 0.f), vk = pk;
#pragma unroll 1
  for (int k = 1; k <= k_hi; ++k) {
    pk = cmul(pk, g.wt);  // w_k^{a t}
    vk = cmul(vk, g.v);   // w_k
    float2 A0 = make_float2(0.f, 0.f), A1 = A0;  // at most 64 entries per thread: their sums stay in fp32
#pragma unroll
    for (int i = 0; i < kDirectRegs; ++i) {
      if (i < g.rows) {
        const float2 tb = ds->tab[i][k];
        A0.x = fmaf(x0[i], tb.x, A0.x);
        A0.y = fmaf(x0[i], tb.y, A0.y);
        A1.x = fmaf(x1[i], tb.x, A1.x);
        A1.y = fmaf(x1[i], tb.y, A1.y);
      }
    }
    for (int i = kDirectRegs; i < g.rows; ++i) {
      const int m = threadIdx.x + kSssThreads * i;
      if (m >= g.M) break;
      const float2 tb = ds->tab[i][k];
      const float xa = x[g.a * m], xb = packed ? x[g.a * m + 1] : 0.f;
      A0.x = fmaf(xa, tb.x, A0.x);
      A0.y = fmaf(xa, tb.y, A0.y);
      A1.x = fmaf(xb, tb.x, A1.x);
      A1.y = fmaf(xb, tb.y, A1.y);
    }
    if (packed) A0 = cadd(A0, cmul(A1, vk));
    float2 F = cmul(A0, pk);
    for (int o = 16; o > 0; o >>= 1) {
      F.x += __shfl_xor_sync(0xffffffffu, F.x, o);
      F.y += __shfl_xor_sync(0xffffffffu, F.y, o);
    }
    if (lane == 0) ds->part[warp][k] = F;
  }
  __syncthreads();
  // warp k adds up bin k over the warps' parts (lane w reads warp w's). (Rolled loops: this runs once, and
  // straight-line code costs more in instruction fetches than its arithmetic takes.)
  if (warp >= 1 && warp <= k_hi) {
    float2 t = ds->part[lane][warp];
#pragma unroll 1
    for (int o = 16; o > 0; o >>= 1) {
      t.x += __shfl_xor_sync(0xffffffffu, t.x, o);
      t.y += __shfl_xor_sync(0xffffffffu, t.y, o);
    }
    if (lane == 0) {
      ds->energy[warp] = static_cast<double>(t.x) * t.x + static_cast<double>(t.y) * t.y;
      ds->bin[warp] = t;
    }
  }
  __syncthreads();
  if (ds->kstar >= 0) return ds->kstar;  // settled in stage 1
  // Stage 3: the first bin at which the cumulative energy reaches the threshold, if it does so clearly
  if (threadIdx.x == 0) {
    const int Kb = n / 2;
    const double thr = ds->tot[1], margin = ds->tot[2];
    int ks = -1;
    double run = 0.0;
#pragma unroll 1
    for (int k = 0; k < kDirectBins; ++k) {
      const double before = run;
      run += ds->energy[k];
      if (run >= thr) {
        if (run >= thr + margin && (k == 0 || before <= thr - margin)) ks = k;
        break;
      }
    }
    if (ks < 0 || ks + T >= kDirectBins || ks + T >= Kb) ks = -1;
    ds->k_hi = ks;
  }
  __syncthreads();
  return ds->k_hi;
}

// The residual mix of every token from the masked bins c_k = mask_k F_k (1 up to k*, raised cosine over the T bins
// after it): y_j = alpha (1/n) [c_0 + 2 sum_k Re(c_k conj(w_k^j))] + (1 - alpha) x_j, written to y (when given) and,
// for the selection, left in buf as order-preserving keys in the layout the transform path leaves them (even n: the
// keys of tokens 2m, 2m + 1 in element m).
__device__ __forceinline__ void direct_apply(const float* __restrict__ x, float* y, int n, bool packed, const DirectGeom& g, int kstar,
                                          int T, float al, bool sel, SkewBuf buf, const DirectSmem* ds) {
  const float om = 1.f - al, c0 = ds->bin[0].x, inv_n = 1.f / static_cast<float>(n);
  const float band = 3.14159265358979f / static_cast<float>(T + 1);
  for (int i0 = 0; i0 < g.rows; i0 += kDirectRegs) {
    float acc0[kDirectRegs], acc1[kDirectRegs];
#pragma unroll
    for (int ii = 0; ii < kDirectRegs; ++ii) acc0[ii] = acc1[ii] = 0.f;
    float2 pk = make_float2(1.f, 0.f), vk = pk;
#pragma unroll 1
    for (int k = 1; k <= kstar + T; ++k) {
      pk = cmul(pk, g.wt);
      vk = cmul(vk, g.v);
      const float mask = k <= kstar ? 1.f : 0.5f * (1.f + __cosf(static_cast<float>(k - kstar) * band));
      const float2 g0 = cscale(cmulc(ds->bin[k], pk), mask);  // c_k conj(w_k^{a t})
      const float2 g1 = cmulc(g0, vk);
#pragma unroll
      for (int ii = 0; ii < kDirectRegs; ++ii) {
        if (i0 + ii < g.rows) {
          const float2 tb = ds->tab[i0 + ii][k];
          acc0[ii] = fmaf(g0.x, tb.x, fmaf(g0.y, tb.y, acc0[ii]));  // Re(g conj(tb))
          acc1[ii] = fmaf(g1.x, tb.x, fmaf(g1.y, tb.y, acc1[ii]));
        }
      }
    }
#pragma unroll
    for (int ii = 0; ii < kDirectRegs; ++ii) {
      const int m = threadIdx.x + kSssThreads * (i0 + ii);
      if (m < g.M) {
        if (packed) {
          const float y0 = fmaf(al, fmaf(2.f, acc0[ii], c0) * inv_n, om * x[2 * m]);
          const float y1 = fmaf(al, fmaf(2.f, acc1[ii], c0) * inv_n, om * x[2 * m + 1]);
          if (y) {
            y[2 * m] = y0;
            y[2 * m + 1] = y1;
          }
          if (sel) buf[m] = make_float2(__uint_as_float(score_key(y0)), __uint_as_float(score_key(y1)));
        } else {
          const float ym = fmaf(al, fmaf(2.f, acc0[ii], c0) * inv_n, om * x[m]);
          if (y) y[m] = ym;
          if (sel) buf[m].x = __uint_as_float(score_key(ym));
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kSssThreads, 1)
sss_kernel(Shape sh, const ReqDesc* __restrict__ reqs, const FftPlan* __restrict__ plans,
           const float2* __restrict__ tables, const float* scores, float* smoothed /* may alias scores */,
           int32_t* __restrict__ kstar_out, float2* __restrict__ scratch, int64_t scratch_per_block,
           const int32_t* __restrict__ order, int n_order, int first_head, const int32_t* __restrict__ budgets,
           const int32_t* __restrict__ cu_kept, int32_t* __restrict__ kept_idx, int* __restrict__ status) {
  extern __shared__ __align__(16) float2 sbuf[];
  __shared__ FftPlan pl;
  __shared__ float2 wp[128];
  __shared__ double red[32];
  __shared__ int s_kstar;
  __shared__ SelectSmem ssm;
  __shared__ DirectSmem dsm;
  // Launched as a programmatic dependent: the block is brought in while the kernel before it drains, reads its plan
  // (written when the plan was made, not by the kernels of the pass), and waits for that kernel only where it first
  // touches the scores.
  chain_release();
  bool waited = false;

  int loaded_plan = -1;  // plan whose tables sit in shared memory
  for (int slot = blockIdx.x; slot < n_order; slot += gridDim.x) {
    const int u = order ? order[slot] : first_head + slot;  // no list: heads first_head, first_head + 1, ...
    if (u < 0) continue;
    const int r = u / sh.heads_per_req;
    const ReqDesc rq = reqs[r];
    __syncthreads();
    if (threadIdx.x == 0) {
      pl = plans[rq.fft_plan];
      s_kstar = 0x7fffffff;
    }
    __syncthreads();
    const int n = pl.n, N = pl.N, Kb = n / 2;
    const SkewBuf buf = pl.in_smem ? SkewBuf{sbuf, 4, 0}
                                   : SkewBuf{scratch + static_cast<int64_t>(blockIdx.x) * scratch_per_block, 31, 0};
    const float* x = scores + rq.score_offset + static_cast<int64_t>(u - rq.head_base) * rq.P;
    float* y = smoothed ? smoothed + rq.score_offset + static_cast<int64_t>(u - rq.head_base) * rq.P : nullptr;

    if (!waited) {
      chain_wait();
      waited = true;
    }
    if (sh.smooth_mode >= AUDIOKV_SMOOTH_AVG_POOL) {
      // Variant: local pooling instead of the spectral filter. The sequence is staged first (scores and smoothed
      // may be the same array), pooled over |i - j| <= pool_kernel / 2 (average: zero padding counts in the
      // divisor; maximum: padding never wins), mixed with alpha and written out; the selection then reads it back.
      float* st = pl.in_smem ? reinterpret_cast<float*>(sbuf)
                             : reinterpret_cast<float*>(scratch + static_cast<int64_t>(blockIdx.x) * scratch_per_block);
      loaded_plan = -1;
      for (int j = threadIdx.x; j < n; j += kSssThreads) st[j] = x[j];
      __syncthreads();
      const int hw = sh.pool_kernel / 2;
      const bool is_max = sh.smooth_mode == AUDIOKV_SMOOTH_MAX_POOL;
      const float inv_pool = 1.f / static_cast<float>(sh.pool_kernel), al = sh.alpha, om = 1.f - sh.alpha;
      for (int j = threadIdx.x; j < n; j += kSssThreads) {
        const int lo = max(0, j - hw), hi = min(n - 1, j + hw);
        float acc = is_max ? -INFINITY : 0.f;
        for (int i = lo; i <= hi; ++i) acc = is_max ? fmaxf(acc, st[i]) : acc + st[i];
        const float pooled = is_max ? acc : acc * inv_pool;
        if (y) y[j] = fmaf(al, pooled, om * st[j]);
      }
      if (threadIdx.x == 0 && kstar_out) kstar_out[u] = 0;
      __syncthreads();
      if (budgets != nullptr) {
        const int P = rq.P, W = sh.window;
        int k = budgets[u] - W;
        if (k < 0 || k > P || y == nullptr) {
          if (threadIdx.x == 0) atomicExch(status, AUDIOKV_EDEVICE);
          k = k < 0 ? 0 : (k > P ? P : k);
        }
        if (y) select_topk([&](int j) -> uint32_t { return score_key(y[j]); }, P, W, k, kept_idx + cu_kept[u], &ssm, status);
      }
      continue;
    }

    const bool sel = budgets != nullptr;
    // A low cut-off is settled from the first few bins of the spectrum, without a transform (see direct_cutoff).
    const bool direct_ok = n >= 4 * kDirectBins && N <= kDirectRows * kSssThreads;
    DirectGeom dg;
    if (direct_ok) dg = direct_geom(n, pl.packed != 0);
    const int kd = direct_ok ? direct_cutoff(x, n, pl.packed != 0, dg, sh.smooth_mode, sh.rho, sh.smooth_kappa,
                                             sh.transition_bins, &dsm)
                             : -1;
    if (kd >= 0) {
      if (threadIdx.x == 0 && kstar_out) kstar_out[u] = kd;
      direct_apply(x, y, n, pl.packed != 0, dg, kd, sh.transition_bins, sh.alpha, sel, buf, &dsm);
    } else {
    // Tables of a direct transform that fit beside the work buffer are staged in shared memory once per plan:
    // the passes read twiddles with data-dependent strides, which from global memory costs a round trip each.
    const float2* tw = tables + pl.seq.tw_offset;
    const float2* post = tables + pl.post_offset;
    const int* pos_tab = reinterpret_cast<const int*>(tables + pl.pos_offset);  // where the forward pass left each bin
    const uint16_t* s_pos = nullptr;
    if (pl.tabs_smem) {
      float2* s_tw = sbuf + sss_padded(N);
      float2* s_post = s_tw + N;
      uint16_t* sp = reinterpret_cast<uint16_t*>(s_post + N / 2 + 1);
      if (loaded_plan != rq.fft_plan) {
        for (int t = threadIdx.x; t < N; t += kSssThreads) {
          s_tw[t] = __ldg(tw + t);
          sp[t] = static_cast<uint16_t>(__ldg(pos_tab + t));
        }
        if (pl.packed)
          for (int t = threadIdx.x; t <= N / 2; t += kSssThreads) s_post[t] = __ldg(post + t);
        loaded_plan = rq.fft_plan;
      }
      tw = s_tw;
      post = s_post;
      s_pos = sp;
    } else {
      loaded_plan = -1;  // this head's work buffer (or its blocks) may run over the staged tables
    }
    // 1. load (packed: z_m = x_2m + i x_2m+1)
    if (pl.packed) {
      for (int m = threadIdx.x; m < N; m += kSssThreads) buf[m] = make_float2(x[2 * m], x[2 * m + 1]);
    } else {
      for (int m = threadIdx.x; m < N; m += kSssThreads) buf[m] = make_float2(x[m], 0.f);
    }
    __syncthreads();

    // 2. forward complex transform; bin k then sits at POS(k)
    if (pl.bluestein)
      bluestein<false>(buf, pl, tables, wp, sbuf, N, pl.half ? Kb + 1 : N, tables + pl.filter_offset);
    else if (pl.in_smem)
      fft_dif(buf, pl.seq, tw, wp);
    else
      fft_dif_big(buf, pl.seq, pl.g_pass, tw, wp, sbuf);
    const bool direct = !pl.bluestein;
#define POS(k) (direct ? (s_pos ? static_cast<int>(s_pos[(k)]) : __ldg(pos_tab + (k))) : (k))

    // 3. packed: turn Z into the real sequence's spectrum F, pairwise in place.
    //    Slot of bin 0 holds (F_0, F_N), both real.
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
          float2 T = cmul(O, post[k]);
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
    const bool no_mean = sh.smooth_mode == AUDIOKV_SMOOTH_ENERGY_NO_MEAN;  // variant: bin 0 adds no energy
    auto energy = [&](int k) -> double {
      if (k == 0 && no_mean) return 0.0;
      if (pl.packed) {
        if (k == 0) return static_cast<double>(buf[0].x) * buf[0].x;
        if (k == N) return static_cast<double>(buf[0].y) * buf[0].y;
      }
      float2 f = buf[POS(k)];
      return static_cast<double>(f.x) * f.x + static_cast<double>(f.y) * f.y;
    };
    if (sh.smooth_mode == AUDIOKV_SMOOTH_FIXED_FRACTION) {
      // variant: the cut-off sits at a fixed fraction of the spectrum, no energies needed
      if (threadIdx.x == 0) s_kstar = static_cast<int>(floor(static_cast<double>(sh.smooth_kappa) * Kb));
    } else {
    // each thread owns `per` consecutive bins; up to 8 of their energies stay in registers for the second look
    double ecache[8];
    double local = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      ecache[i] = k0 + i < k1 ? energy(k0 + i) : 0.0;
      local += ecache[i];
    }
    for (int k = k0 + 8; k < k1; ++k) local += energy(k);
    const double before = block_excl_scan(local, red);
    const double total = block_sum(local, red);
    const double thr = static_cast<double>(sh.rho) * total;
    {
      double run = before;
      bool found = false;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (!found && k0 + i < k1) {
          run += ecache[i];
          if (run >= thr) {
            atomicMin(&s_kstar, k0 + i);
            found = true;
          }
        }
      }
      for (int k = k0 + 8; k < k1 && !found; ++k) {
        run += energy(k);
        if (run >= thr) {
          atomicMin(&s_kstar, k);
          found = true;
        }
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
          float2 O = cmulc(Tt, post[k]);
          float2 iO = mul_i(O);
          buf[pk] = cadd(E, iO);
          buf[pq] = cconj(csub(E, iO));
        }
      }
    } else if (pl.half) {
      // bins 0 .. Kb alone go back: x_j = (2 / N) Re sum_{k <= Kb} h_k e^{+2 pi i j k / N}, h_0 = F_0 / 2, h_k = F_k
      for (int k = threadIdx.x; k <= Kb; k += kSssThreads) buf[k] = cscale(buf[k], k == 0 ? 0.5f * weight(0) : weight(k));
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
      bluestein<true>(buf, pl, tables, wp, sbuf, pl.half ? Kb + 1 : N, N,
                      tables + (pl.half ? pl.filter2_offset : pl.filter_offset));
    else if (pl.in_smem)
      fft_dit_inv(buf, pl.seq, tw, wp);
    else
      fft_dit_inv_big(buf, pl.seq, pl.g_pass, tw, wp, sbuf);
#undef POS

    // 7. residual mix. `smoothed` (optional) gets the result; when budgets are given the result
    //    also stays in the work buffer, as order-preserving keys, for the selection below.
    const float inv = (pl.half ? 2.f : 1.f) / static_cast<float>(N), al = sh.alpha, om = 1.f - sh.alpha;
    // packed: the keys of tokens 2m and 2m+1 replace element m; otherwise the key of token m goes to the real part of element m
    if (pl.packed) {
      for (int m = threadIdx.x; m < N; m += kSssThreads) {
        float2 z = buf[m];
        const float x0 = x[2 * m], x1 = x[2 * m + 1];
        const float y0 = fmaf(al, z.x * inv, om * x0), y1 = fmaf(al, z.y * inv, om * x1);
        if (y) {
          y[2 * m] = y0;
          y[2 * m + 1] = y1;
        }
        if (sel) buf[m] = make_float2(__uint_as_float(score_key(y0)), __uint_as_float(score_key(y1)));
      }
    } else {
      for (int m = threadIdx.x; m < N; m += kSssThreads) {
        const float ym = fmaf(al, buf[m].x * inv, om * x[m]);
        if (y) y[m] = ym;
        if (sel) buf[m].x = __uint_as_float(score_key(ym));
      }
    }
    }  // transform path
    if (sel) {
      // 8. top-k of the smoothed scores, straight from the work buffer
      const int P = rq.P, W = sh.window;
      int k = budgets[u] - W;
      if (k < 0 || k > P) {
        if (threadIdx.x == 0) atomicExch(status, AUDIOKV_EDEVICE);
        k = k < 0 ? 0 : P;
      }
      __syncthreads();
      if (pl.packed)
        select_topk([&](int j) -> uint32_t { const float2 e = buf[j >> 1]; return __float_as_uint((j & 1) ? e.y : e.x); }, P, W, k,
                    kept_idx + cu_kept[u], &ssm, status);
      else
        select_topk([&](int j) -> uint32_t { return __float_as_uint(buf[j].x); }, P, W, k, kept_idx + cu_kept[u], &ssm, status);
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
    // Wrapped conjugate chirp b[d] = exp(+i pi d^2 / N) at position d for index differences d = out - in >= 0 and at
    // M - |d| for d < 0, zero elsewhere. Full plan: |d| < N both ways. Half plan: the forward filter serves d in
    // [-(N-1), Kb] (N inputs, Kb + 1 outputs), the inverse one d in [-Kb, N-1].
    const int Kb = (pl.n - 1) / 2;
    const int pos_f = pl.half ? Kb + 1 : N, neg_f = N;       // forward filter: d in (-neg_f, pos_f)
    const int pos_i = N, neg_i = pl.half ? Kb + 1 : N;       // inverse filter (half plans only)
    auto chirp_at = [&](int d) -> float2 {  // exp(+i pi d^2 / N), the exponent reduced exactly
      const long long q = (static_cast<long long>(d) * d) % (2LL * N);
      double s, c;
      sincospi(static_cast<double>(q) / N, &s, &c);
      return make_float2(static_cast<float>(c), static_cast<float>(s));
    };
    for (int j = gid; j < M; j += gsz) {
      if (j < N) {
        const float2 b = chirp_at(j);
        tables[pl.chirp_offset + j] = make_float2(b.x, -b.y);
      }
      // position j holds difference +j inside the positive support, difference -(M - j) inside the negative one
      // (they never collide: M is at least their total length), zero in between
      auto wrapped = [&](int pos, int neg) -> float2 {
        if (j < pos) return chirp_at(j);
        if (M - j < neg) return chirp_at(M - j);
        return make_float2(0.f, 0.f);
      };
      tables[pl.filter_offset + j] = wrapped(pos_f, neg_f);
      if (pl.half) tables[pl.filter2_offset + j] = wrapped(pos_i, neg_i);
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
  for (int which = 0; which < (pl.half ? 2 : 1); ++which) {
    float2* f = tables + (which ? pl.filter2_offset : pl.filter_offset);
    __syncthreads();
    fft_dif(SkewBuf{f, 31, 0}, pl.seq, tables + pl.seq.tw_offset, wp);
    const float inv = 1.f / static_cast<float>(pl.M);
    for (int j = threadIdx.x; j < pl.M; j += kSssThreads) f[j] = cscale(f[j], inv);
  }
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
                       int64_t scratch_per_block, int grid, size_t smem_bytes, const int32_t* order, int n_order,
                       int first_head, const int32_t* budgets, const int32_t* cu_kept, int32_t* kept_idx, int* status,
                       Launch ln) {
  cudaError_t e = cudaFuncSetAttribute(sss_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  e = launch_chained(sss_kernel, dim3(grid), dim3(kSssThreads), smem_bytes, ln.stream, sh, d_reqs, d_plans, d_tables, scores,
                     smoothed, kstar, scratch, scratch_per_block, order, n_order, first_head, budgets, cu_kept, kept_idx,
                     status);
  ln.done(budgets ? "sss_select" : "sss");
  return e;
}

}  // namespace akv
