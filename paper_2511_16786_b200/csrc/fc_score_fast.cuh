// Specialised kernels of the three transform passes for power-of-two sequence
// lengths N = N1*N2 with N1 = 16*R1B and N2 = 16*R2B (R1B, R2B in {2,4,8,16}),
// i.e. N from 1024 to 65536.  Same mathematics as the generic kernels in
// fc_score.cu (see the header comment there); what differs is the mapping:
//
//  * every thread owns two adjacent channels (one float4 = two complex values),
//    so all shared-memory and workspace accesses are 128-bit and a twiddle is
//    loaded once for two butterflies;
//  * a thread keeps a whole radix-16 butterfly (16 points x 2 channels) in
//    registers; the first stage of pass 1 is fed straight from the K/V rows in
//    global memory and the last stage of each pass is written straight to global
//    memory, so a tile crosses shared memory once per exchange;
//  * all strides are compile-time constants.
//
// The transform is left unnormalised (factor N); pass 3 folds 1/N^2 into the score.
#pragma once
#include "fc_common.cuh"

namespace fast {

__device__ __forceinline__ int perm_token(int p, int N) {
  const int half = (N + 1) >> 1;
  return p < half ? 2 * p : 2 * (N - 1 - p) + 1;
}

// two adjacent channels of one row
template <typename T> struct Load2;
template <> struct Load2<float> {
  __device__ static float2 ld(const float *p) { return __ldg(reinterpret_cast<const float2 *>(p)); }
};
template <> struct Load2<__half> {
  __device__ static float2 ld(const __half *p) {
    const unsigned u = __ldg(reinterpret_cast<const unsigned *>(p));
    return __half22float2(*reinterpret_cast<const __half2 *>(&u));
  }
};
template <> struct Load2<__nv_bfloat16> {
  __device__ static float2 ld(const __nv_bfloat16 *p) {
    const unsigned u = __ldg(reinterpret_cast<const unsigned *>(p));
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
  }
};

// exp(+j*pi*n*n/N), the chirp of the convolution form of an N-point DFT; n*n is reduced modulo 2N
// (one period) in integers first.  Costs a 64-bit division: the passes read it from a table (k_chirp_tables).
// 4-byte asynchronous copy global -> shared (two 16-bit channels), and the wait for this thread's copies
__device__ __forceinline__ void cp_async4(void *smem_dst, const void *gsrc) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ float2 pair16_to_float2(unsigned u, const __half *) {
  return __half22float2(*reinterpret_cast<const __half2 *>(&u));
}
__device__ __forceinline__ float2 pair16_to_float2(unsigned u, const __nv_bfloat16 *) {
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}
__device__ __forceinline__ float2 pair16_to_float2(unsigned, const float *) { return make_float2(0.f, 0.f); }

// exp(-2*pi*j*r/n) for table lengths the master table has no entries for (not a power of two)
__device__ __forceinline__ float2 root_of_unity(int r, int n) {
  double sn, cs;
  sincospi(-2.0 * (double)r / (double)n, &sn, &cs);
  return make_float2((float)cs, (float)sn);
}

__device__ __forceinline__ float2 chirp_f(int n, int N) {
  const unsigned long long r = ((unsigned long long)n * (unsigned long long)n) % (2ull * (unsigned long long)N);
  float s, c;
  sincospif(__fdiv_rn((float)(unsigned)r, (float)N), &s, &c);
  return make_float2(c, s);
}

// tab[n] = chirp(n), tab[N + q] = exp(j*pi*q/N) for n, q = 0..N-1: what the chirp modes of passes 1 and 3 need per
// row, computed once per sequence length instead of once per thread and row.
__global__ void k_chirp_tables(float2 *__restrict__ tab, int N) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  tab[i] = chirp_f(i, N);
  float sn, cs;
  sincospif(__fdiv_rn((float)i, (float)N), &sn, &cs);
  tab[N + i] = make_float2(cs, sn);
}

// What pass 1 transforms.
//   LD_KV     : the K/V rows of a power-of-two sequence (N = N1*N2 points).
//   LD_CHIRP  : chirp convolution, first half: the N < N1*N2 rows times conj(chirp), zeros behind them.
//   LD_FILTER : chirp convolution, second half: the N-point spectrum spec[q][col] through the low-pass
//               residual filter, conjugated (an inverse DFT is the conjugate of the forward DFT of the
//               conjugate) and times conj(chirp), zeros behind.
//   LD_BAND   : as LD_FILTER for the band form of the chirp path: spec holds only the 2*band+1 bins q = -band..band
//               of the N-point spectrum (row q + band); the input is conj(Wb[q]) * conj(chirp(q)) with the low-pass
//               part Wb[q] = (W[q] + exp(j*pi*q/N) W[-q]) / 2 (one formula for both signs of q and for q = 0),
//               zeros behind.  `omega` carries the band.
//   LD_KERNEL : the chirp kernel of the convolution itself in column 0 (other columns zero), wrapped to the transform
//               length: chirp(|n|) for |n| < N, or for the band form (`omega` carries the band, else -1)
//               chirp(|n - band|) for n = -(N-1) .. 2*band.
enum { LD_KV = 0, LD_CHIRP = 1, LD_FILTER = 2, LD_BAND = 3, LD_KERNEL = 4 };
// What pass 2 does between its forward and inverse halves: the DCT/low-pass residual filter on paired rows,
// or a multiplication by the spectrum of the chirp kernel (rows 2x and 2x+1, unrelated).  MID_CONV2 is the
// convolution for rows of 2*N2 points: the two halves of the block take the even and the odd samples of ONE
// row through N2-point transforms, a radix-2 step joins them before the multiplication and splits the
// product again after it (bins k and k + N2 live in the two halves' threads of equal index).
enum { MID_FILTER = 0, MID_CONV = 1, MID_CONV2 = 2 };
// What pass 3 does with the rows it gets back: scores of a power-of-two sequence, the N-point spectrum of
// the chirp path (rows < N times conj(chirp)), or the scores at the end of the chirp path.
// OUT_SCORE_BAND: end of the band form: the rows are N times the conjugate of the Base KV (low-pass part) in the
// reordered domain; the K/V rows are read again and the score is |z - z_base|^2.
enum { OUT_SCORE = 0, OUT_SPEC = 1, OUT_SCORE_CHIRP = 2, OUT_SCORE_BAND = 3 };

// x[p] *= w^p (CONJ: conj(w)^p), p = 1..15, for both channels, from w and w^4 alone: the other powers are products of
// at most three table values (w^p = w^(4g) * w^r), which replaces 13 of 15 shared-memory reads per use by arithmetic.
template <bool CONJ>
__device__ __forceinline__ void twiddle_powers16(float2 (&x0)[16], float2 (&x1)[16], float2 c1, float2 c4) {
  if (CONJ) { c1.y = -c1.y; c4.y = -c4.y; }
  const float2 c2 = cmul(c1, c1), c3 = cmul(c2, c1);
  float2 base = c4;
  x0[1] = cmul(x0[1], c1); x1[1] = cmul(x1[1], c1);
  x0[2] = cmul(x0[2], c2); x1[2] = cmul(x1[2], c2);
  x0[3] = cmul(x0[3], c3); x1[3] = cmul(x1[3], c3);
#pragma unroll
  for (int g = 1; g < 4; ++g) {
    const float2 b1 = cmul(base, c1), b2 = cmul(base, c2), b3 = cmul(base, c3);
    x0[4 * g] = cmul(x0[4 * g], base);     x1[4 * g] = cmul(x1[4 * g], base);
    x0[4 * g + 1] = cmul(x0[4 * g + 1], b1); x1[4 * g + 1] = cmul(x1[4 * g + 1], b1);
    x0[4 * g + 2] = cmul(x0[4 * g + 2], b2); x1[4 * g + 2] = cmul(x1[4 * g + 2], b2);
    x0[4 * g + 3] = cmul(x0[4 * g + 3], b3); x1[4 * g + 3] = cmul(x1[4 * g + 3], b3);
    if (g < 3) base = cmul(base, c4);
  }
}

// x[p] *= b * s^p (CONJ: the conjugate of that), p = 0..15, from b, s and s^4.
template <bool CONJ>
__device__ __forceinline__ void twiddle_affine16(float2 (&x0)[16], float2 (&x1)[16], float2 b, float2 s1, float2 s4) {
  if (CONJ) { b.y = -b.y; s1.y = -s1.y; s4.y = -s4.y; }
  const float2 s2 = cmul(s1, s1), s3 = cmul(s2, s1);
  float2 base = b;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const float2 b1 = cmul(base, s1), b2 = cmul(base, s2), b3 = cmul(base, s3);
    x0[4 * g] = cmul(x0[4 * g], base);     x1[4 * g] = cmul(x1[4 * g], base);
    x0[4 * g + 1] = cmul(x0[4 * g + 1], b1); x1[4 * g + 1] = cmul(x1[4 * g + 1], b1);
    x0[4 * g + 2] = cmul(x0[4 * g + 2], b2); x1[4 * g + 2] = cmul(x1[4 * g + 2], b2);
    x0[4 * g + 3] = cmul(x0[4 * g + 3], b3); x1[4 * g + 3] = cmul(x1[4 * g + 3], b3);
    if (g < 3) base = cmul(base, s4);
  }
}

template <int R>
__device__ __forceinline__ void dft_fwd(float2 (&x)[R]) { dft_small<R, -1>(x); }
template <int R>
__device__ __forceinline__ void dft_inv(float2 (&x)[R]) { dft_small<R, +1>(x); }

// ---------------------------------------------------------------------------
// pass 1: grid (N2, group columns / (2*CPW)), block CPW*R1B.
// Thread (cp = tid % CPW, j = tid / CPW): channels 2cp, 2cp+1 of the slice; first
// stage points n1 = j + R1B*p, p = 0..A-1, loaded from the K/V rows.  N1 = A*R1B: A = 16 with R1B = 2..16 for
// power-of-two lengths, A = 10, 12 or 14 with R1B = 16 for the chirp path's lengths 2^a * {5, 3, 7}.
// ---------------------------------------------------------------------------
// Launch bounds: three resident blocks of 256 threads (80 registers), the measured best for the power-of-two path.
template <typename T, int R1B, int CPW, int LD = LD_KV, int A = 16>
__global__ void __launch_bounds__(CPW * R1B, (768 / (CPW * R1B)) > 0 ? 768 / (CPW * R1B) : 1)
k_p1(const T *__restrict__ k, const T *__restrict__ v, long long stride_token, long long stride_head,
     int head0, int head_dim, int N, int N2, int ncol_ws, float2 *__restrict__ ws,
     const float2 *__restrict__ master, int master_len, double *__restrict__ partial,
     const float2 *__restrict__ spec = nullptr, int omega = 0, const float2 *__restrict__ ctab = nullptr) {
  // ctab (chirp modes): ctab[n] = chirp(n) and ctab[N + q] = exp(j*pi*q/N), n, q = 0..N-1
  constexpr int N1 = A * R1B, NT = CPW * R1B, IT = (A + R1B - 1) / R1B, NW = (NT + 31) / 32;
  extern __shared__ float4 smem4[];
  float4 *S = smem4;                                        // [N1][CPW]
  float2 *tw = reinterpret_cast<float2 *>(S + N1 * CPW);    // [N1]
  __shared__ double red[2][NW];
  const int tid = threadIdx.x, cp = tid % CPW, j = tid / CPW;
  const int n2 = blockIdx.x, gc0 = blockIdx.y * (2 * CPW);
  const int h = head0 + gc0 / head_dim, c = gc0 % head_dim + 2 * cp;
  const T *kb = k + (long long)h * stride_head + c;
  const T *vb = v + (long long)h * stride_head + c;

  __shared__ float2 cts[LD == LD_CHIRP ? N1 : 1];           // chirp of row n1 of this block (position n1*N2 + n2)
  if (LD == LD_CHIRP) {
    for (int i = tid; i < N1; i += NT) {
      const int n = i * N2 + n2;
      cts[i] = n < N ? __ldg(ctab + n) : make_float2(1.f, 0.f);
    }
  }
  float2 x0[A], x1[A];
  float accK = 0.f, accV = 0.f;
#pragma unroll
  for (int p = 0; p < A; ++p) {
    const int n = (j + R1B * p) * N2 + n2;
    if (LD == LD_KV) {
      const long long off = (long long)perm_token(n, N) * stride_token;
      const float2 kk = Load2<T>::ld(kb + off), vv = Load2<T>::ld(vb + off);
      x0[p] = make_float2(kk.x, vv.x);
      x1[p] = make_float2(kk.y, vv.y);
    } else if (LD == LD_CHIRP) {
      // loads only (rows past the sequence read row 0 and are zeroed): the sums of squares and the rotation by the
      // conjugate chirp follow the barrier, with the chirp factors of this block's rows in shared memory by then
      const long long off = (long long)perm_token(n < N ? n : 0, N) * stride_token;
      const float2 kk = Load2<T>::ld(kb + off), vv = Load2<T>::ld(vb + off);
      const float keep = n < N ? 1.f : 0.f;
      x0[p] = make_float2(kk.x * keep, vv.x * keep);
      x1[p] = make_float2(kk.y * keep, vv.y * keep);
    } else if (LD == LD_KERNEL) {
      x0[p] = x1[p] = make_float2(0.f, 0.f);
      if (gc0 == 0 && cp == 0) {
        const int M = N1 * N2, band = omega;
        int a = -1;                                  // argument of the chirp; -1: outside the kernel's support
        if (band < 0) {
          if (n < N) a = n;
          else if (n > M - N) a = M - n;
        } else {
          if (n <= 2 * band) a = n < band ? band - n : n - band;
          else if (n > M - N) a = band + (M - n);
        }
        if (a >= 0) x0[p] = chirp_f(a, N);
      }
    } else if (LD == LD_BAND) {
      x0[p] = x1[p] = make_float2(0.f, 0.f);
      const int band = omega;
      if (n <= 2 * band) {
        const int q = n - band, aq = q < 0 ? -q : q;
        const float4 P4 = __ldcg(reinterpret_cast<const float4 *>(spec + (size_t)n * ncol_ws + gc0 + 2 * cp));
        const float4 Q4 = __ldcg(reinterpret_cast<const float4 *>(spec + (size_t)(2 * band - n) * ncol_ws + gc0 + 2 * cp));
        float2 u = __ldg(ctab + N + aq);                         // exp(j*pi*q/N)
        if (q < 0) u.y = -u.y;
        const float2 ch = __ldg(ctab + aq);
        const float2 W0 = cscale(cadd(make_float2(P4.x, P4.y), cmul(make_float2(Q4.x, Q4.y), u)), 0.5f);
        const float2 W1 = cscale(cadd(make_float2(P4.z, P4.w), cmul(make_float2(Q4.z, Q4.w), u)), 0.5f);
        x0[p] = cmul_conj(cconj(W0), ch);
        x1[p] = cmul_conj(cconj(W1), ch);
      }
    } else {
      x0[p] = x1[p] = make_float2(0.f, 0.f);
      if (n < N) {
        const int q = n, qp = (N - q) % N;
        const float4 P4 = __ldcg(reinterpret_cast<const float4 *>(spec + (size_t)q * ncol_ws + gc0 + 2 * cp));
        const float4 Q4 = __ldcg(reinterpret_cast<const float4 *>(spec + (size_t)qp * ncol_ws + gc0 + 2 * cp));
        const float2 u = __ldg(ctab + N + q);
        const float inL = (q <= omega) ? 0.5f : 0.f;
        const float inH = (q != 0 && N - q <= omega) ? 0.5f : 0.f;
        const float2 ch = __ldg(ctab + n);
        const float2 P0 = make_float2(P4.x, P4.y), P1 = make_float2(P4.z, P4.w);
        const float2 uQ0 = cmul(make_float2(Q4.x, Q4.y), u), uQ1 = cmul(make_float2(Q4.z, Q4.w), u);
        float2 E0 = csub(csub(P0, cscale(cadd(P0, uQ0), inL)), cscale(csub(P0, uQ0), inH));
        float2 E1 = csub(csub(P1, cscale(cadd(P1, uQ1), inL)), cscale(csub(P1, uQ1), inH));
        x0[p] = cmul_conj(cconj(E0), ch);
        x1[p] = cmul_conj(cconj(E1), ch);
      }
    }
  }
  for (int i = tid; i < N1; i += NT) tw[i] = (A == 16) ? master[(size_t)i * (master_len / N1)] : root_of_unity(i, N1);
  __syncthreads();
  if (LD == LD_KV || LD == LD_CHIRP) {
#pragma unroll
    for (int p = 0; p < A; ++p) {
      accK = fmaf(x0[p].x, x0[p].x, fmaf(x1[p].x, x1[p].x, accK));
      accV = fmaf(x0[p].y, x0[p].y, fmaf(x1[p].y, x1[p].y, accV));
    }
  }
  if (LD == LD_CHIRP) {
#pragma unroll
    for (int p = 0; p < A; ++p) {
      const float2 ch = cts[j + R1B * p];
      x0[p] = cmul_conj(x0[p], ch);
      x1[p] = cmul_conj(x1[p], ch);
    }
  }
  dft_fwd<A>(x0);
  dft_fwd<A>(x1);
#pragma unroll
  for (int p = 0; p < A; ++p) {
    if (p > 0) {
      const float2 w = tw[j * p];
      x0[p] = cmul(x0[p], w);
      x1[p] = cmul(x1[p], w);
    }
    S[(j + R1B * p) * CPW + cp] = make_float4(x0[p].x, x0[p].y, x1[p].x, x1[p].y);
  }
  __syncthreads();
  // second stage: radix R1B inside sub-block pp; bin k1 = pp + 16*q
#pragma unroll
  for (int it = 0; it < IT; ++it) {
    const int pp = j + R1B * it;
    if (A % R1B != 0 && pp >= A) break;
    float2 y0[R1B], y1[R1B];
#pragma unroll
    for (int q = 0; q < R1B; ++q) {
      const float4 t = S[(q + R1B * pp) * CPW + cp];
      y0[q] = make_float2(t.x, t.y);
      y1[q] = make_float2(t.z, t.w);
    }
    dft_fwd<R1B>(y0);
    dft_fwd<R1B>(y1);
#pragma unroll
    for (int q = 0; q < R1B; ++q) {
      const int k1 = pp + A * q;
      float4 *dst = reinterpret_cast<float4 *>(ws + ((size_t)k1 * N2 + n2) * ncol_ws + gc0 + 2 * cp);
      *dst = make_float4(y0[q].x, y0[q].y, y1[q].x, y1[q].y);
    }
  }
  if (LD == LD_FILTER || LD == LD_BAND || LD == LD_KERNEL) return;
  // per-block sums of squares (total energy of Eq. 12, by Parseval)
  const double a = warp_sum_d((double)accK), b = warp_sum_d((double)accV);
  if ((tid & 31) == 0) { red[0][tid >> 5] = a; red[1][tid >> 5] = b; }
  __syncthreads();
  if (tid == 0) {
    double sa = 0, sb = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) { sa += red[0][i]; sb += red[1][i]; }
    const size_t slot = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
    partial[2 * slot] = sa;
    partial[2 * slot + 1] = sb;
  }
}

// ---------------------------------------------------------------------------
// pass 2: grid (N1/2, group columns / (2*CP)) for the filter and the plain convolution, (N1, ...) for MID_CONV2; block 2*CP*R2B.
// Thread (cp = tid % CP, hf = (tid / CP) & 1, j = tid / (2*CP)): channel pair cp of
// the slice, half hf (k1 = blockIdx.x or N1 - blockIdx.x), first-stage points
// n2 = j + R2B*p.
// ---------------------------------------------------------------------------
template <int R2B, int CP, int MID = MID_FILTER>
__global__ void __launch_bounds__(2 * CP * R2B, 512 / (2 * CP * R2B > 32 ? 2 * CP * R2B : 32))
k_p2(int N1, int ncol_ws, float2 *__restrict__ ws, const float2 *__restrict__ master, int master_len,
     int omega, const float2 *__restrict__ hhat = nullptr, float scale = 1.f, int hrev = 0,
     float2 *__restrict__ hout = nullptr) {
  // hrev (convolution variants): multiply by the spectrum of the index-reversed kernel, hhat[(-bin) mod N]
  // hout (convolution variants): forward half only; the spectrum of column 0 goes to hout[bin] (the chirp kernel's
  // spectrum for transform lengths the generic kernels do not take)
  constexpr int N2 = 16 * R2B, NT = 2 * CP * R2B, IT = 16 / R2B;
  extern __shared__ float4 smem4[];
  float4 *S = smem4;                                         // [2][N2][CP]
  float2 *tw = reinterpret_cast<float2 *>(S + 2 * N2 * CP);  // [N2]   w_N2^i
  // tables with one part per half: the second half starts H2 = N2 + 4 entries in, so that threads of the two halves
  // reading the same index hit different banks
  constexpr int H2 = N2 + 4;
  float2 *twN = tw + N2;                                     // [2][N2] w_N^(n2*k1)
  float2 *uT = twN + H2 + N2;                                // [2][N2] exp(-j*pi*(k1 + N1*k2)/N)
  float2 *hs = uT + H2 + N2;                                  // [2][N2] convolution variants: scaled kernel spectrum of this block's bins
  const int tid = threadIdx.x, cp = tid % CP, hf = (tid / CP) & 1, j = tid / (2 * CP);
  // MID_CONV: grid.x = N1/2, the two halves of the block are the unrelated rows 2x and 2x + 1
  const int k1a = (MID == MID_CONV) ? 2 * blockIdx.x : blockIdx.x;
  // MID_FILTER: grid.x = N1/2; block x > 0 holds the partner rows x and N1 - x, block 0 the two rows that are their
  // own partners, 0 and N1/2 (each half then reads its partner bins from itself)
  const int k1b = (MID == MID_CONV) ? 2 * blockIdx.x + 1
                : (MID == MID_CONV2) ? (int)blockIdx.x : (k1a == 0 ? N1 / 2 : N1 - k1a);
  const bool self = (MID == MID_FILTER) && (k1a == 0);
  const int k1 = hf ? k1b : k1a;
  constexpr int ROW = (MID == MID_CONV2) ? 2 * N2 : N2;      // points of one row of the workspace
  const int N = N1 * ROW;
  const int gc0 = blockIdx.y * (2 * CP);
  constexpr bool active = true;

  {
    // N is a power of two (every root is in the master table) or, on the chirp path, 2^a * {3, 5, 7}
    const bool tab = (master_len % N) == 0;
    const int mstepN = tab ? master_len / N : 0, ustep = master_len / (2 * N);
    for (int i = tid; i < N2; i += NT) {
      tw[i] = master[(size_t)i * (master_len / N2)];
      if (MID == MID_CONV2) {
        const int ra = ((2 * i) * k1a) % N, rb = ((2 * i + 1) * k1a) % N;
        twN[i] = tab ? master[(size_t)ra * mstepN] : root_of_unity(ra, N);        // even samples: n2 = 2i
        twN[H2 + i] = tab ? master[(size_t)rb * mstepN] : root_of_unity(rb, N);   // odd samples: n2 = 2i + 1
        uT[i] = master[(size_t)i * (master_len / ROW)];                          // w_ROW^k of the radix-2 step
      } else if (MID == MID_CONV) {
        const int ra = (i * k1a) % N, rb = (i * k1b) % N;
        twN[i] = tab ? master[(size_t)ra * mstepN] : root_of_unity(ra, N);
        twN[H2 + i] = tab ? master[(size_t)rb * mstepN] : root_of_unity(rb, N);
      } else {
        twN[i] = master[(size_t)((i * k1a) & (N - 1)) * mstepN];
        twN[H2 + i] = master[(size_t)((i * k1b) & (N - 1)) * mstepN];
      }
      if (MID == MID_FILTER) {
        uT[i] = master[(size_t)(k1a + N1 * i) * ustep];
        uT[H2 + i] = master[(size_t)(k1b + N1 * i) * ustep];
      }
      if ((MID == MID_CONV || MID == MID_CONV2) && hout == nullptr) {
        // bins of the two halves: rows k1a and k1b (MID_CONV) or the lower and upper half of row k1a (MID_CONV2)
        const int ba = k1a + N1 * i, bb = (MID == MID_CONV2) ? k1a + N1 * (i + N2) : k1b + N1 * i;
        hs[i] = cscale(__ldg(hhat + ((hrev && ba != 0) ? N - ba : ba)), scale);
        hs[H2 + i] = cscale(__ldg(hhat + ((hrev && bb != 0) ? N - bb : bb)), scale);
      }
    }
  }
  float4 *Sh = S + hf * (N2 * CP);
  // row twiddles: entry j + R2B*p of this half's table is entry j times the p-th power of a step that the table
  // holds at R2B (MID_CONV2: both halves belong to one row, the step sits in the even samples' table)
  const int so = (MID == MID_CONV2) ? 0 : hf * H2;
  float2 x0[16], x1[16];
  // element n2 of the row: MID_CONV2 interleaves the halves (n2 = 2i + hf)
  float2 *base = ws + ((size_t)k1 * ROW + (MID == MID_CONV2 ? hf : 0)) * ncol_ws + gc0 + 2 * cp;
  const size_t rstride = (size_t)(MID == MID_CONV2 ? 2 : 1) * ncol_ws;
  if (active) {
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float4 t = __ldcg(reinterpret_cast<const float4 *>(base + (size_t)(j + R2B * p) * rstride));
      x0[p] = make_float2(t.x, t.y);
      x1[p] = make_float2(t.z, t.w);
    }
  }
  __syncthreads();
  if (active) {
    twiddle_affine16<false>(x0, x1, twN[hf * H2 + j], twN[so + R2B], twN[so + 4 * R2B]);
    dft_fwd<16>(x0);
    dft_fwd<16>(x1);
    twiddle_powers16<false>(x0, x1, tw[j], tw[4 * j]);
#pragma unroll
    for (int p = 0; p < 16; ++p)
      Sh[(j + R2B * p) * CP + cp] = make_float4(x0[p].x, x0[p].y, x1[p].x, x1[p].y);
  }
  __syncthreads();
  // second forward stage, written back in place (each sub-block is touched by one thread only);
  // registers keep bins k2 = pp + 16*q at index it*R2B + q
  if (active) {
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
      float2 y0[R2B], y1[R2B];
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        const float4 t = Sh[(q + R2B * pp) * CP + cp];
        y0[q] = make_float2(t.x, t.y);
        y1[q] = make_float2(t.z, t.w);
      }
      dft_fwd<R2B>(y0);
      dft_fwd<R2B>(y1);
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        x0[it * R2B + q] = y0[q];
        x1[it * R2B + q] = y1[q];
        // MID_CONV keeps its bins in registers: nobody else reads them, and the rows of this sub-block are written
        // again only by this thread (first inverse stage), so neither the store nor the two barriers are needed
        // MID_FILTER: only bins inside the two bands are read by their partners (the partner of an in-band bin is
        // in the other band), so the rest, 1 - 2*gamma of them, is not written back
        bool wanted = (MID != MID_CONV);
        if (MID == MID_FILTER) {
          const int bin = k1 + N1 * (pp + 16 * q);
          wanted = bin <= omega || N - bin <= omega;
        }
        if (wanted) Sh[(q + R2B * pp) * CP + cp] = make_float4(y0[q].x, y0[q].y, y1[q].x, y1[q].y);
      }
    }
  }
  if (MID != MID_CONV) __syncthreads();       // full spectra of both halves are in shared memory
  if (active) {
    const float4 *Sp = S + (self ? hf : 1 - hf) * (N2 * CP);
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        const int k2 = pp + 16 * q;
        const int bin = k1 + N1 * k2;
        if (MID == MID_CONV) {
          if (hout != nullptr) {
            if (cp == 0 && blockIdx.y == 0) hout[bin] = x0[it * R2B + q];
            continue;
          }
          const float2 hq = hs[hf * H2 + k2];
          x0[it * R2B + q] = cmul(x0[it * R2B + q], hq);
          x1[it * R2B + q] = cmul(x1[it * R2B + q], hq);
          continue;
        }
        if (MID == MID_CONV2) {
          // this thread holds E[k2] (hf = 0) or O[k2] (hf = 1); A[k2] = E + w O, A[k2 + N2] = E - w O
          const float4 t = Sp[(q + R2B * pp) * CP + cp];
          const float2 w = uT[k2];
          float2 &m0 = x0[it * R2B + q], &m1 = x1[it * R2B + q];
          const float2 e0 = hf ? make_float2(t.x, t.y) : m0, e1 = hf ? make_float2(t.z, t.w) : m1;
          const float2 o0 = cmul(hf ? m0 : make_float2(t.x, t.y), w), o1 = cmul(hf ? m1 : make_float2(t.z, t.w), w);
          const int binh = k1 + N1 * (k2 + hf * N2);
          if (hout != nullptr) {
            if (cp == 0 && blockIdx.y == 0) hout[binh] = hf ? csub(e0, o0) : cadd(e0, o0);
            continue;
          }
          const float2 hq = hs[hf * H2 + k2];
          m0 = cmul(hf ? csub(e0, o0) : cadd(e0, o0), hq);
          m1 = cmul(hf ? csub(e1, o1) : cadd(e1, o1), hq);
          continue;
        }
        const bool inL = bin <= omega, inH = (N - bin) <= omega;
        float2 &P0 = x0[it * R2B + q], &P1 = x1[it * R2B + q];
        if (bin == 0 || (inL && inH)) {
          P0 = make_float2(0.f, 0.f);
          P1 = make_float2(0.f, 0.f);
        } else if (inL || inH) {
          const int k2p = (k1 == 0) ? ((N2 - k2) & (N2 - 1)) : (N2 - 1 - k2);
          const float4 t = Sp[((k2p >> 4) + R2B * (k2p & 15)) * CP + cp];
          float2 u = uT[hf * H2 + k2];                             // exp(-j*pi*bin/N)
          const float sgn = inL ? -0.5f : 0.5f;                   // E = (P -/+ uQ)/2 with u = exp(+j*pi*bin/N)
          u = make_float2(u.x * sgn, -u.y * sgn);
          const float2 q0 = make_float2(t.x, t.y), q1 = make_float2(t.z, t.w);
          P0 = make_float2(fmaf(q0.x, u.x, fmaf(-q0.y, u.y, 0.5f * P0.x)),
                           fmaf(q0.x, u.y, fmaf(q0.y, u.x, 0.5f * P0.y)));
          P1 = make_float2(fmaf(q1.x, u.x, fmaf(-q1.y, u.y, 0.5f * P1.x)),
                           fmaf(q1.x, u.y, fmaf(q1.y, u.x, 0.5f * P1.y)));
        }
      }
    }
  }
  if ((MID == MID_CONV || MID == MID_CONV2) && hout != nullptr) return;
  if (MID == MID_CONV2) {
    // B[k2] sits in half 0, B[k2 + N2] in half 1: even samples come back from B_lo + B_hi, odd samples from
    // (B_lo - B_hi) * conj(w)
    __syncthreads();                                   // everyone has read its partner's spectrum
#pragma unroll
    for (int it = 0; it < IT; ++it)
#pragma unroll
      for (int q = 0; q < R2B; ++q)
        Sh[(q + R2B * (j + R2B * it)) * CP + cp] = make_float4(x0[it * R2B + q].x, x0[it * R2B + q].y,
                                                               x1[it * R2B + q].x, x1[it * R2B + q].y);
    __syncthreads();
    const float4 *Sp = S + (1 - hf) * (N2 * CP);
#pragma unroll
    for (int it = 0; it < IT; ++it)
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        const int pp = j + R2B * it, k2 = pp + 16 * q;
        const float4 t = Sp[(q + R2B * pp) * CP + cp];
        float2 &m0 = x0[it * R2B + q], &m1 = x1[it * R2B + q];
        if (hf == 0) {
          m0 = cadd(m0, make_float2(t.x, t.y));
          m1 = cadd(m1, make_float2(t.z, t.w));
        } else {
          const float2 w = uT[k2];
          m0 = cmul_conj(csub(make_float2(t.x, t.y), m0), w);
          m1 = cmul_conj(csub(make_float2(t.z, t.w), m1), w);
        }
      }
  }
  if (active) {
    // first inverse stage (mirror of the second forward stage)
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      float2 y0[R2B], y1[R2B];
#pragma unroll
      for (int q = 0; q < R2B; ++q) { y0[q] = x0[it * R2B + q]; y1[q] = x1[it * R2B + q]; }
      dft_inv<R2B>(y0);
      dft_inv<R2B>(y1);
#pragma unroll
      for (int q = 0; q < R2B; ++q) { x0[it * R2B + q] = y0[q]; x1[it * R2B + q] = y1[q]; }
    }
  }
  if (MID != MID_CONV) __syncthreads();       // all partner reads are done
  if (active) {
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
#pragma unroll
      for (int q = 0; q < R2B; ++q)
        Sh[(q + R2B * pp) * CP + cp] = make_float4(x0[it * R2B + q].x, x0[it * R2B + q].y,
                                                  x1[it * R2B + q].x, x1[it * R2B + q].y);
    }
  }
  __syncthreads();
  if (active) {
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float4 t = Sh[(j + R2B * p) * CP + cp];
      x0[p] = make_float2(t.x, t.y);
      x1[p] = make_float2(t.z, t.w);
    }
    twiddle_powers16<true>(x0, x1, tw[j], tw[4 * j]);
    dft_inv<16>(x0);
    dft_inv<16>(x1);
    twiddle_affine16<true>(x0, x1, twN[hf * H2 + j], twN[so + R2B], twN[so + 4 * R2B]);
#pragma unroll
    for (int p = 0; p < 16; ++p)
      *reinterpret_cast<float4 *>(base + (size_t)(j + R2B * p) * rstride) =
          make_float4(x0[p].x, x0[p].y, x1[p].x, x1[p].y);
  }
}

// ---------------------------------------------------------------------------
// pass 3: grid (N2, heads of the group), block CPW*R1B.  Inverse DFT over k1,
// squared magnitude summed over the channels of the head, scores and the
// per-block outlier-energy partial sums.
// ---------------------------------------------------------------------------
// OUT_SPEC and OUT_SCORE_CHIRP: N is the sequence length (< N1*N2), rows at or past it are dropped;
// OUT_SPEC stores to spec[row][col] and returns; OUT_SCORE_CHIRP is given done_counter == nullptr and
// leaves the final energy sums to the caller.
// band >= 0 (band form of the chirp path): OUT_SPEC keeps rows 0 .. 2*band (bin q = row - band, rotated by
// conj(chirp(|q|))); OUT_SCORE_BAND reads the K/V rows again (kin/vin: first token of the sequence, first channel of
// the column group) and scores |z - z_base|^2 with z_base = conj(row * conj(chirp)) / N.
template <int R1B, int CPW, int OUT = OUT_SCORE, typename T = float, int A = 16>
__global__ void __launch_bounds__(CPW * R1B, 512 / (CPW * R1B))
k_p3(int N, int N2, int ncol_ws, const float2 *__restrict__ ws, const float2 *__restrict__ master,
     int master_len, float *__restrict__ scores, int head0, int head_dim, long long score_stride,
     float inv_scale, double *__restrict__ partial, unsigned *__restrict__ done_counter,
     unsigned total_blocks, const double *__restrict__ part_tot, int n_tot,
     const double *__restrict__ part_hi, int n_hi, double *__restrict__ energy,
     float2 *__restrict__ spec = nullptr, float energy_scale = 0.f, int accumulate = 0, int band = -1,
     const T *__restrict__ kin = nullptr, const T *__restrict__ vin = nullptr, long long stride_token = 0,
     long long stride_head = 0, const float2 *__restrict__ ctab = nullptr) {
  // OUT_SCORE_CHIRP with a head transformed in column groups: head_dim is the group's width, energy_scale the
  // head's true channel count, and every group after the first adds to the stored score (accumulate).
  constexpr int N1 = A * R1B, NT = CPW * R1B, IT = (A + R1B - 1) / R1B, NW = (NT + 31) / 32;
  extern __shared__ float4 smem4[];
  float4 *S = smem4;                                        // [N1][CPW]
  float2 *tw = reinterpret_cast<float2 *>(S + N1 * CPW);    // [N1]
  // band form, 16-bit inputs: the K/V rows the residual is taken against are copied asynchronously into
  // stg[2*A][NT] (this thread's slots only) while the two inverse stages run
  constexpr bool STAGE = (OUT == OUT_SCORE_BAND) && sizeof(T) == 2;
  unsigned *stg = reinterpret_cast<unsigned *>(tw + N1);
  __shared__ double red[2][NW];
  const int tid = threadIdx.x, cp = tid % CPW, j = tid / CPW;
  const int n2 = blockIdx.x, hh = blockIdx.y;
  for (int i = tid; i < N1; i += NT) tw[i] = (A == 16) ? master[(size_t)i * (master_len / N1)] : root_of_unity(i, N1);
  // chirp factor of each row of this block (row n1 is position n1*N2 + n2), visible after the first barrier
  __shared__ float2 cts[OUT != OUT_SCORE ? N1 : 1];
  if (OUT != OUT_SCORE) {
    for (int i = tid; i < N1; i += NT) {
      const int pos = i * N2 + n2;
      const bool spec_band = (OUT == OUT_SPEC && band >= 0);
      const bool valid = spec_band ? pos <= 2 * band : pos < N;
      const int cpos = spec_band ? (pos < band ? band - pos : pos - band) : pos;
      cts[i] = valid ? __ldg(ctab + cpos) : make_float2(0.f, 0.f);
    }
  }

  float acc[16];            // |residual|^2 of rows j + R1B*p summed over this thread's channels (K and V)
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 0.f;
  float totK = 0.f, totV = 0.f;

  const int nslices = head_dim / (2 * CPW);
  for (int sl = 0; sl < nslices; ++sl) {
    const int gc0 = hh * head_dim + sl * (2 * CPW);
    if (STAGE) {
      const int col = gc0 + 2 * cp;
      const long long coff = (long long)(head0 + col / head_dim) * stride_head + col % head_dim;
#pragma unroll
      for (int p = 0; p < A; ++p) {
        const int pos = (j + R1B * p) * N2 + n2;
        if (pos < N) {
          const long long off = (long long)perm_token(pos, N) * stride_token + coff;
          cp_async4(stg + (2 * p) * NT + tid, kin + off);
          cp_async4(stg + (2 * p + 1) * NT + tid, vin + off);
        }
      }
    }
    // inverse radix-R1B stage on bins k1 = pp + 16*q, straight from the workspace
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
      if (A % R1B != 0 && pp >= A) break;
      float2 y0[R1B], y1[R1B];
#pragma unroll
      for (int q = 0; q < R1B; ++q) {
        const float4 t = __ldcg(reinterpret_cast<const float4 *>(
            ws + ((size_t)(pp + A * q) * N2 + n2) * ncol_ws + gc0 + 2 * cp));
        y0[q] = make_float2(t.x, t.y);
        y1[q] = make_float2(t.z, t.w);
      }
      dft_inv<R1B>(y0);
      dft_inv<R1B>(y1);
#pragma unroll
      for (int q = 0; q < R1B; ++q)
        S[(q + R1B * pp) * CPW + cp] = make_float4(y0[q].x, y0[q].y, y1[q].x, y1[q].y);
    }
    __syncthreads();
    float2 x0[A], x1[A];
#pragma unroll
    for (int p = 0; p < A; ++p) {
      const float4 t = S[(j + R1B * p) * CPW + cp];
      x0[p] = make_float2(t.x, t.y);
      x1[p] = make_float2(t.z, t.w);
      if (p > 0) {
        const float2 w = tw[j * p];
        x0[p] = cmul_conj(x0[p], w);
        x1[p] = cmul_conj(x1[p], w);
      }
    }
    dft_inv<A>(x0);
    dft_inv<A>(x1);
    if (STAGE) cp_async_wait_all();
#pragma unroll
    for (int p = 0; p < A; ++p) {
      if (OUT != OUT_SCORE) {
        const int pos = (j + R1B * p) * N2 + n2;
        if (OUT == OUT_SPEC && band >= 0) {
          if (pos > 2 * band) continue;
        } else if (pos >= N) {
          continue;
        }
        const float2 ch = cts[j + R1B * p];                      // chirp of this row
        x0[p] = cmul_conj(x0[p], ch);
        x1[p] = cmul_conj(x1[p], ch);
        if (OUT == OUT_SPEC) {
          *reinterpret_cast<float4 *>(spec + (size_t)pos * ncol_ws + gc0 + 2 * cp) =
              make_float4(x0[p].x, x0[p].y, x1[p].x, x1[p].y);
          continue;
        }
        if (OUT == OUT_SCORE_BAND) {
          // residual against the input rows: z_base = conj(x) / N (inv_scale carries 1/d only)
          float2 kk, vv;
          if (STAGE) {
            kk = pair16_to_float2(stg[(2 * p) * NT + tid], kin);
            vv = pair16_to_float2(stg[(2 * p + 1) * NT + tid], vin);
          } else {
            const int col = gc0 + 2 * cp;
            const long long off = (long long)perm_token(pos, N) * stride_token +
                                  (long long)(head0 + col / head_dim) * stride_head + col % head_dim;
            kk = Load2<T>::ld(kin + off);
            vv = Load2<T>::ld(vin + off);
          }
          const float rn = 1.f / (float)N;
          x0[p] = make_float2(fmaf(-x0[p].x, rn, kk.x), fmaf(x0[p].y, rn, vv.x));
          x1[p] = make_float2(fmaf(-x1[p].x, rn, kk.y), fmaf(x1[p].y, rn, vv.y));
        }
      }
      const float ek = fmaf(x0[p].x, x0[p].x, x1[p].x * x1[p].x);
      const float ev = fmaf(x0[p].y, x0[p].y, x1[p].y * x1[p].y);
      totK += ek;
      totV += ev;
      acc[p] += ek + ev;
    }
    __syncthreads();
  }
  if (OUT == OUT_SPEC) return;
  // transposed reduction over the CPW lanes that share j: the 16 row sums are halved at every
  // step until one is left, further steps are plain adds; row p = cp >> log2(CPW/16)
  {
    int count = 16;
#pragma unroll
    for (int s = CPW / 2; s >= 1; s >>= 1) {
      if (count > 1) {
        const int half = count / 2;
#pragma unroll
        for (int i = 0; i < half; ++i) {
          const bool up = (cp & s) != 0;
          const float send = up ? acc[i] : acc[i + half];
          const float keep = up ? acc[i + half] : acc[i];
          acc[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
        count = half;
      } else {
        acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], s);
      }
    }
  }
  constexpr int DUP = CPW / 16;                             // lanes that end with the same row sum
  if ((cp & (DUP - 1)) == 0 && cp / DUP < A) {            // rows A..15 of the reduction are padding
    const int p = (j + R1B * (cp / DUP)) * N2 + n2;
    if (OUT == OUT_SCORE) {
      scores[(long long)(head0 + hh) * score_stride + perm_token(p, N)] = acc[0] * inv_scale;
    } else if (p < N) {
      float *dst = scores + (long long)(head0 + hh) * score_stride + perm_token(p, N);
      *dst = accumulate ? *dst + acc[0] * inv_scale : acc[0] * inv_scale;
    }
  }
  const double dk = warp_sum_d((double)(totK * inv_scale));
  const double dv = warp_sum_d((double)(totV * inv_scale));
  if ((tid & 31) == 0) { red[0][tid >> 5] = dk; red[1][tid >> 5] = dv; }
  __syncthreads();
  if (tid == 0) {
    double sa = 0, sb = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) { sa += red[0][i]; sb += red[1][i]; }
    const size_t slot = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
    const double es = (OUT == OUT_SCORE_CHIRP || OUT == OUT_SCORE_BAND) ? (double)energy_scale : (double)head_dim;
    partial[2 * slot] = sa * es;
    partial[2 * slot + 1] = sb * es;
  }
  // The last block of the sequence (over all head groups, on either stream) adds up the
  // per-block partial sums in a fixed order: energy = (hiK, totK, hiV, totV).
  if (OUT == OUT_SCORE_CHIRP || OUT == OUT_SCORE_BAND) return;
  __shared__ bool is_last;
  if (tid == 0) {
    __threadfence();
    const unsigned prev = atomicAdd(done_counter, 1u);
    is_last = (prev + 1u == total_blocks);
    if (is_last) *done_counter = 0u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  double *redd = reinterpret_cast<double *>(smem4);        // [4][NT], the tile is no longer needed
  double a0 = 0, a1 = 0, b0 = 0, b1 = 0;
  for (int i = tid; i < n_tot; i += NT) { a0 += __ldcg(part_tot + 2 * i); a1 += __ldcg(part_tot + 2 * i + 1); }
  for (int i = tid; i < n_hi; i += NT) { b0 += __ldcg(part_hi + 2 * i); b1 += __ldcg(part_hi + 2 * i + 1); }
  redd[tid] = b0; redd[NT + tid] = a0; redd[2 * NT + tid] = b1; redd[3 * NT + tid] = a1;
  __syncthreads();
  for (int st = NT / 2; st > 0; st >>= 1) {
    if (tid < st)
      for (int q = 0; q < 4; ++q) redd[q * NT + tid] += redd[q * NT + tid + st];
    __syncthreads();
  }
  if (tid < 4) energy[tid] = redd[tid * NT];
}

}  // namespace fast
