// fc_score_layer: Outlier KV Recognition Module (Sec. 3.2.1, Eq. 5-10) plus the
// energy sums of Eq. 11-12, for one layer.
//
// How the score is computed.  For one head, channel c, the complex sequence
// z[i] = K[i,c] + j V[i,c] carries both matrices through one transform (the DCT is a
// real linear map, so real and imaginary parts never mix).  The orthonormal DCT-II of
// Eq. 6-7 of a length-N sequence equals Re(exp(-j*pi*m/(2N)) * W[m]) * alpha[m], where W
// is the N-point DFT of the even/odd reordering  w[n] = z[2n], w[N-1-n] = z[2n+1].
// Low-pass filtering (Eq. 8) and the inverse DCT (Eq. 9) are linear, so the
// spectrum of the residual  z - z_base  in that DFT domain is, with P = W[q],
// Q = W[N-q], u = exp(j*pi*q/N):
//     E[q] = P - [q <= omega] (P + uQ)/2 - [N-q <= omega] (P - uQ)/2,   E[0] = 0,
// and the residual itself is the inverse DFT of E.  Dev[x] (Eq. 10) is then
// (1/d) * sum_c |residual|^2 with the real part belonging to K and the imaginary
// part to V; K and V are read exactly once and no Base KV is ever stored.
//
// The N-point DFT is done in three passes over an intermediate that stays in L2
// (N = N1*N2, n = n1*N2 + n2, q = k1 + N1*k2):
//   pass 1  for every n2: DFT over n1                      -> A[k1][n2]
//   pass 2  for every k1 (with N1-k1, which holds the partner bins N-q):
//           twiddle, DFT over n2, the filter above, inverse DFT over k2, twiddle -> B[k1][n2]
//   pass 3  for every n2: inverse DFT over k1, |.|^2 summed over the channels -> scores
// Lengths that are not a power of two (or are below 16) go through Bluestein's
// chirp convolution on a power-of-two length M >= 2N-1 with the same three passes.
#include "fc_common.cuh"
#include "fc_score_fast.cuh"

#include <math.h>
#include <mutex>
#include <type_traits>
#include <unordered_map>

namespace {

constexpr int kThreads = 256;

// ---------------------------------------------------------------------------
// index helpers
// ---------------------------------------------------------------------------
// Reordered index p -> token (w[n] = z[2n] for n < ceil(N/2), w[N-1-n] = z[2n+1]).
__device__ __forceinline__ int perm_token(int p, int N) {
  const int half = (N + 1) >> 1;
  return p < half ? 2 * p : 2 * (N - 1 - p) + 1;
}

// exp(j*pi*n^2/N), the Bluestein chirp; the phase is reduced exactly in integers.
__device__ __forceinline__ float2 chirp(int n, int N) {
  const unsigned long long r = ((unsigned long long)n * (unsigned long long)n) % (2ull * (unsigned long long)N);
  float s, c;
  sincospif(__fdiv_rn((float)(unsigned)r, (float)N), &s, &c);
  return make_float2(c, s);
}

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int VEC = 4;
  __device__ static void load(const float *p, float (&out)[4]) {
    const float4 v = *reinterpret_cast<const float4 *>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Elem<__half> {
  static constexpr int VEC = 8;
  __device__ static void load(const __half *p, float (&out)[8]) {
    const uint4 v = *reinterpret_cast<const uint4 *>(p);
    const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 f = __half22float2(h[i]); out[2 * i] = f.x; out[2 * i + 1] = f.y; }
  }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int VEC = 8;
  __device__ static void load(const __nv_bfloat16 *p, float (&out)[8]) {
    const uint4 v = *reinterpret_cast<const uint4 *>(p);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); out[2 * i] = f.x; out[2 * i + 1] = f.y; }
  }
};

// ---------------------------------------------------------------------------
// pass-1 loaders: value of transform input p for VEC consecutive workspace columns
// ---------------------------------------------------------------------------
// K/V rows of one sequence.  Column gc of the group maps to head h0 + gc/d, channel gc%d.
template <typename T, bool BLUE>
struct KvLoader {
  static constexpr int VEC = Elem<T>::VEC;
  const T *k, *v;          // already offset to the first token of the sequence
  long long stride_token, stride_head;
  int head0, head_dim, N;
  float accK, accV;        // running sums of squares (per thread)
  __device__ void init() { accK = 0.f; accV = 0.f; }
  __device__ void load(int p, int gc, float2 (&out)[VEC]) {
    if (BLUE && p >= N) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) out[i] = make_float2(0.f, 0.f);
      return;
    }
    const int t = perm_token(p, N);
    const int h = head0 + gc / head_dim, c = gc % head_dim;
    const long long off = (long long)t * stride_token + (long long)h * stride_head + c;
    float a[VEC], b[VEC];
    Elem<T>::load(k + off, a);
    Elem<T>::load(v + off, b);
#pragma unroll
    for (int i = 0; i < VEC; ++i) { accK = fmaf(a[i], a[i], accK); accV = fmaf(b[i], b[i], accV); }
    if (BLUE) {
      const float2 ch = chirp(p, N);
#pragma unroll
      for (int i = 0; i < VEC; ++i) out[i] = cmul_conj(make_float2(a[i], b[i]), ch);
    } else {
#pragma unroll
      for (int i = 0; i < VEC; ++i) out[i] = make_float2(a[i], b[i]);
    }
  }
};

// Bluestein, second half: reads the N-point spectrum W[q][col], applies the
// low-pass residual filter, and feeds conj(E[q]) * conj(chirp) to the forward
// machinery (an inverse DFT is the conjugate of the forward DFT of the conjugate).
struct FilterLoader {
  static constexpr int VEC = 2;
  const float2 *spec;      // [N][ncol]
  int ncol, N, omega;
  __device__ void init() {}
  __device__ void load(int p, int gc, float2 (&out)[2]) {
    if (p >= N) { out[0] = out[1] = make_float2(0.f, 0.f); return; }
    const int q = p, qp = (N - q) % N;
    const float4 P4 = *reinterpret_cast<const float4 *>(spec + (size_t)q * ncol + gc);
    const float4 Q4 = *reinterpret_cast<const float4 *>(spec + (size_t)qp * ncol + gc);
    float s, c;
    sincospif(__fdiv_rn((float)q, (float)N), &s, &c);
    const float2 u = make_float2(c, s);
    const float inL = (q <= omega) ? 0.5f : 0.f;
    const float inH = (q != 0 && N - q <= omega) ? 0.5f : 0.f;
    const float2 ch = chirp(p, N);
    const float2 Pv[2] = {make_float2(P4.x, P4.y), make_float2(P4.z, P4.w)};
    const float2 Qv[2] = {make_float2(Q4.x, Q4.y), make_float2(Q4.z, Q4.w)};
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float2 uQ = cmul(Qv[i], u);
      float2 E = Pv[i];
      E = csub(E, cscale(cadd(Pv[i], uQ), inL));
      E = csub(E, cscale(csub(Pv[i], uQ), inH));
      out[i] = cmul_conj(cconj(E), ch);
    }
  }
};

// Bluestein convolution kernel h[p] = chirp(|p|) wrapped to length M, in column 0.
// band >= 0: the kernel of the band form, g[j] = chirp(|j - band|) for j = -(N-1) .. 2*band, wrapped (outputs
// 0 .. 2*band of the convolution are the bins -band .. band; needs M >= N + 2*band).
struct ChirpKernelLoader {
  static constexpr int VEC = 2;
  int N, M, band;
  __device__ void init() {}
  __device__ void load(int p, int gc, float2 (&out)[2]) {
    out[0] = out[1] = make_float2(0.f, 0.f);
    if (gc != 0) return;
    if (band < 0) {
      if (p < N) out[0] = chirp(p, N);
      else if (p > M - N) out[0] = chirp(M - p, N);
    } else {
      if (p <= 2 * band) out[0] = chirp(p < band ? band - p : p - band, N);
      else if (p > M - N) out[0] = chirp(band + (M - p), N);
    }
  }
};

// ---------------------------------------------------------------------------
// pass 1: DFT over n1 for one n2 and one slice of cs columns
// grid (N2, ncol_ws/cs)
// ---------------------------------------------------------------------------
template <class Loader>
__global__ void __launch_bounds__(kThreads)
k_pass1(Loader ld, FftPlan plan, int N2, int ncol_ws, int cs_log2, float2 *__restrict__ ws,
        const float2 *__restrict__ master, int master_len, double *__restrict__ partial) {
  extern __shared__ float2 smem[];
  const int N1 = plan.len, cs = 1 << cs_log2;
  float2 *S = smem;
  float2 *tw = S + (size_t)N1 * cs;
  int *rev = reinterpret_cast<int *>(tw + N1);
  const int tid = threadIdx.x;
  const int n2 = blockIdx.x, gc0 = blockIdx.y * cs;

  for (int i = tid; i < N1; i += kThreads) {
    tw[i] = master[(size_t)i * (master_len / N1)];
    rev[i] = digit_rev(plan, i);
  }
  ld.init();
  constexpr int VEC = Loader::VEC;
  const int vec_per_row = cs / VEC;
  for (int it = tid; it < N1 * vec_per_row; it += kThreads) {
    const int row = it / vec_per_row, cv = it - row * vec_per_row;
    float2 vals[VEC];
    ld.load(row * N2 + n2, gc0 + cv * VEC, vals);
    float2 *dst = S + (size_t)row * cs + cv * VEC;
#pragma unroll
    for (int i = 0; i < VEC; i += 2)
      *reinterpret_cast<float4 *>(dst + i) = make_float4(vals[i].x, vals[i].y, vals[i + 1].x, vals[i + 1].y);
  }
  __syncthreads();
  fft_forward_tile(plan, S, cs_log2, tw, tid, kThreads);
  for (int w = tid; w < N1 * cs; w += kThreads) {
    const int pos = w >> cs_log2, c = w & (cs - 1);
    ws[((size_t)rev[pos] * N2 + n2) * ncol_ws + gc0 + c] = S[w];
  }
  if constexpr (!std::is_same<Loader, FilterLoader>::value && !std::is_same<Loader, ChirpKernelLoader>::value) {
    if (partial != nullptr) {
      __shared__ double red[2][kThreads / 32];
      double a = warp_sum_d((double)ld.accK), b = warp_sum_d((double)ld.accV);
      if ((tid & 31) == 0) { red[0][tid >> 5] = a; red[1][tid >> 5] = b; }
      __syncthreads();
      if (tid == 0) {
        double sa = 0, sb = 0;
        for (int i = 0; i < kThreads / 32; ++i) { sa += red[0][i]; sb += red[1][i]; }
        const size_t slot = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
        partial[2 * slot] = sa;
        partial[2 * slot + 1] = sb;
      }
    }
  }
}

// ---------------------------------------------------------------------------
// pass 2: for one k1 (and its partner N1-k1): twiddle, DFT over n2, middle step,
// inverse DFT over k2, twiddle, scale.  In place in the workspace.
// MID_DCT   : low-pass residual filter between bins q and N-q   grid (N1/2+1, ncol_ws/cs2)
// MID_MULH  : pointwise product with the chirp spectrum          grid (N1, ncol_ws/cs2)
// MID_SPEC  : forward only; column 0 written to hhat[k]          grid (N1, 1)
// ---------------------------------------------------------------------------
enum { MID_DCT = 0, MID_MULH = 1, MID_SPEC = 2 };

template <int MID>
__global__ void __launch_bounds__(kThreads)
k_pass2(FftPlan plan, int N1, int ncol_ws, int cs2_log2, float2 *__restrict__ ws,
        const float2 *__restrict__ master, int master_len, int omega,
        float2 *__restrict__ hhat, float scale) {
  extern __shared__ float2 smem[];
  const int N2 = plan.len, cs2 = 1 << cs2_log2;
  const int Nfft = N1 * N2;
  const int tid = threadIdx.x;
  int k1a = blockIdx.x, k1b = blockIdx.x;
  int halves = 1;
  if (MID == MID_DCT) {
    k1b = (N1 - k1a) % N1;
    halves = (k1b != k1a) ? 2 : 1;
  }
  const int ncolT_log2 = cs2_log2 + (halves - 1);
  const int ncolT = 1 << ncolT_log2;
  const int gc0 = blockIdx.y * cs2;

  float2 *S = smem;                                    // [N2][2*cs2] for the paired rows of MID_DCT, else [N2][cs2]
  float2 *tw = S + (size_t)N2 * (MID == MID_DCT ? 2 : 1) * cs2;   // [N2]
  float2 *twN = tw + N2;                               // [2][N2]
  unsigned short *rev = reinterpret_cast<unsigned short *>(twN + 2 * N2);   // [N2]
  unsigned short *pos_of = rev + N2;                                       // [N2]

  const int mstepN = master_len / Nfft;
  for (int i = tid; i < N2; i += kThreads) {
    tw[i] = master[(size_t)i * (master_len / N2)];
    twN[i] = master[(size_t)(((long long)i * k1a) % Nfft) * mstepN];
    twN[N2 + i] = master[(size_t)(((long long)i * k1b) % Nfft) * mstepN];
    const int k = digit_rev(plan, i);
    rev[i] = (unsigned short)k;
    pos_of[k] = (unsigned short)i;
  }
  __syncthreads();

  // load with the forward inter-pass twiddle w_N^(n2*k1)
  for (int w = tid; w < N2 * ncolT; w += kThreads) {
    const int n2 = w >> ncolT_log2, col = w & (ncolT - 1);
    const int hf = col >> cs2_log2, c = col & (cs2 - 1);
    const int k1 = hf ? k1b : k1a;
    const float2 a = ws[((size_t)k1 * N2 + n2) * ncol_ws + gc0 + c];
    S[w] = cmul(a, twN[hf * N2 + n2]);
  }
  __syncthreads();
  fft_forward_tile(plan, S, ncolT_log2, tw, tid, kThreads);

  if (MID == MID_SPEC) {
    for (int pos = tid; pos < N2; pos += kThreads)
      hhat[k1a + N1 * (int)rev[pos]] = S[(size_t)pos << ncolT_log2];
    return;
  }
  if (MID == MID_MULH) {
    for (int w = tid; w < N2 * ncolT; w += kThreads) {
      const int pos = w >> ncolT_log2;
      S[w] = cmul(S[w], hhat[k1a + N1 * (int)rev[pos]]);
    }
  } else {
    // Every pair {q, N-q} is owned by the thread that meets the smaller bin.
    const int N = Nfft;
    const int ustep = master_len / (2 * N);
    for (int w = tid; w < N2 * ncolT; w += kThreads) {
      const int pos = w >> ncolT_log2, col = w & (ncolT - 1);
      const int hf = col >> cs2_log2, c = col & (cs2 - 1);
      const int k1 = hf ? k1b : k1a;
      const int q = k1 + N1 * (int)rev[pos];
      const int qp = (N - q) % N;
      if (q > qp) continue;
      const int k1p = qp % N1, k2p = qp / N1;
      const int hfp = (k1p == k1) ? hf : 1 - hf;
      const int wp = ((int)pos_of[k2p] << ncolT_log2) + (hfp << cs2_log2) + c;
      const float2 P = S[w], Q = S[wp];
      if (q == 0) { S[w] = make_float2(0.f, 0.f); continue; }
      const float2 u = cconj(master[(size_t)q * ustep]);           // exp(+j*pi*q/N)
      const float2 uQ = cmul(Q, u);
      const float inLq = (q <= omega) ? 0.5f : 0.f, inHq = (N - q <= omega) ? 0.5f : 0.f;
      float2 Eq = P;
      Eq = csub(Eq, cscale(cadd(P, uQ), inLq));
      Eq = csub(Eq, cscale(csub(P, uQ), inHq));
      S[w] = Eq;
      if (qp != q) {
        // bin N-q: u' = exp(j*pi*(N-q)/N) = -conj(u)
        const float2 upP = cscale(cmul_conj(P, u), -1.f);
        const float inLp = (qp <= omega) ? 0.5f : 0.f, inHp = (q <= omega) ? 0.5f : 0.f;
        float2 Ep = Q;
        Ep = csub(Ep, cscale(cadd(Q, upP), inLp));
        Ep = csub(Ep, cscale(csub(Q, upP), inHp));
        S[wp] = Ep;
      }
    }
  }
  __syncthreads();
  fft_inverse_tile(plan, S, ncolT_log2, tw, tid, kThreads);
  for (int w = tid; w < N2 * ncolT; w += kThreads) {
    const int n2 = w >> ncolT_log2, col = w & (ncolT - 1);
    const int hf = col >> cs2_log2, c = col & (cs2 - 1);
    const int k1 = hf ? k1b : k1a;
    const float2 r = cscale(cmul_conj(S[w], twN[hf * N2 + n2]), scale);
    ws[((size_t)k1 * N2 + n2) * ncol_ws + gc0 + c] = r;
  }
}

// ---------------------------------------------------------------------------
// pass 3: inverse DFT over k1 for one n2.
// EPI_SCORE : loops over the head's column slices, accumulates sum_c |.|^2 per row,
//             writes scores and the per-block outlier-energy partials.  grid (N2, heads)
// EPI_SPEC  : multiplies by conj(chirp) and stores rows p < N of the N-point
//             spectrum to spec[p][col] (Bluestein, first half).    grid (N2, ncol_ws/cs)
// ---------------------------------------------------------------------------
enum { EPI_SCORE = 0, EPI_SPEC = 1 };

template <int EPI, bool BLUE>
__global__ void __launch_bounds__(kThreads)
k_pass3(FftPlan plan, int N2, int N, int ncol_ws, int cs_log2, const float2 *__restrict__ ws,
        const float2 *__restrict__ master, int master_len,
        float2 *__restrict__ spec, float *__restrict__ scores, int head0, int head_dim,
        long long score_stride, float inv_scale, double *__restrict__ partial,
        float energy_scale, int accumulate) {
  // EPI_SCORE sums the head_dim columns starting at blockIdx.y * head_dim; when a head is
  // transformed in several column groups, head_dim is the group width, energy_scale the
  // true number of channels, and every group after the first adds to the stored score.
  extern __shared__ float2 smem[];
  const int N1 = plan.len, cs = 1 << cs_log2;
  float2 *S = smem;
  float2 *tw = S + (size_t)N1 * cs;
  int *rev = reinterpret_cast<int *>(tw + N1);
  float *accK = reinterpret_cast<float *>(rev + N1);
  float *accV = accK + N1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n2 = blockIdx.x;

  for (int i = tid; i < N1; i += kThreads) {
    tw[i] = master[(size_t)i * (master_len / N1)];
    rev[i] = digit_rev(plan, i);
    accK[i] = 0.f;
    accV[i] = 0.f;
  }
  __syncthreads();

  const int nslices = (EPI == EPI_SCORE) ? head_dim / cs : 1;
  for (int sl = 0; sl < nslices; ++sl) {
    const int gc0 = (EPI == EPI_SCORE) ? (blockIdx.y * head_dim + sl * cs) : blockIdx.y * cs;
    for (int w = tid; w < N1 * cs; w += kThreads) {
      const int pos = w >> cs_log2, c = w & (cs - 1);
      S[w] = ws[((size_t)rev[pos] * N2 + n2) * ncol_ws + gc0 + c];
    }
    __syncthreads();
    fft_inverse_tile(plan, S, cs_log2, tw, tid, kThreads);
    if (EPI == EPI_SPEC) {
      for (int w = tid; w < N1 * cs; w += kThreads) {
        const int n1 = w >> cs_log2, c = w & (cs - 1);
        const int p = n1 * N2 + n2;
        if (p < N) spec[(size_t)p * ncol_ws + gc0 + c] = cmul_conj(S[w], chirp(p, N));
      }
    } else {
      for (int n1 = warp; n1 < N1; n1 += kThreads / 32) {
        const int p = n1 * N2 + n2;
        float sk = 0.f, sv = 0.f;
        if (!BLUE || p < N) {
          float2 ch = make_float2(1.f, 0.f);
          if (BLUE) ch = chirp(p, N);
          for (int c = lane; c < cs; c += 32) {
            float2 e = S[((size_t)n1 << cs_log2) + c];
            if (BLUE) e = cmul_conj(e, ch);
            sk = fmaf(e.x, e.x, sk);
            sv = fmaf(e.y, e.y, sv);
          }
        }
        sk = warp_sum(sk);
        sv = warp_sum(sv);
        if (lane == 0) { accK[n1] += sk; accV[n1] += sv; }
      }
    }
    __syncthreads();
  }

  if (EPI == EPI_SCORE) {
    const int h = head0 + blockIdx.y;
    double dk = 0.0, dv = 0.0;
    for (int n1 = tid; n1 < N1; n1 += kThreads) {
      const int p = n1 * N2 + n2;
      if (p < N) {
        const float k = accK[n1] * inv_scale, v = accV[n1] * inv_scale;   // already divided by d
        float *dst = scores + (long long)h * score_stride + perm_token(p, N);
        *dst = accumulate ? *dst + (k + v) : k + v;
        dk += (double)k;
        dv += (double)v;
      }
    }
    __shared__ double red[2][kThreads / 32];
    dk = warp_sum_d(dk);
    dv = warp_sum_d(dv);
    if (lane == 0) { red[0][warp] = dk; red[1][warp] = dv; }
    __syncthreads();
    if (tid == 0) {
      double sa = 0, sb = 0;
      for (int i = 0; i < kThreads / 32; ++i) { sa += red[0][i]; sb += red[1][i]; }
      const size_t slot = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
      partial[2 * slot] = sa * (double)energy_scale;      // d * sum Dev_k = outlier-band energy
      partial[2 * slot + 1] = sb * (double)energy_scale;
    }
  }
}

// Fixed-order reduction of the per-block partial sums of one sequence into
// energy[4] = (hiK, totK, hiV, totV).  One block.
__global__ void __launch_bounds__(256)
k_energy_finalize(const double *__restrict__ part_tot, int n_tot, const double *__restrict__ part_hi,
                  int n_hi, double *__restrict__ energy) {
  __shared__ double red[4][256];
  const int tid = threadIdx.x;
  double a0 = 0, a1 = 0, b0 = 0, b1 = 0;
  for (int i = tid; i < n_tot; i += 256) { a0 += part_tot[2 * i]; a1 += part_tot[2 * i + 1]; }
  for (int i = tid; i < n_hi; i += 256) { b0 += part_hi[2 * i]; b1 += part_hi[2 * i + 1]; }
  red[0][tid] = b0; red[1][tid] = a0; red[2][tid] = b1; red[3][tid] = a1;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (tid < s)
      for (int j = 0; j < 4; ++j) red[j][tid] += red[j][tid + s];
    __syncthreads();
  }
  if (tid < 4) energy[tid] = red[tid][0];
}

// ---------------------------------------------------------------------------
// Power spectrum of a layer (Eq. 11): P_k[m], P_v[m] = sum over heads and channels of C[m,c]^2.
// With z = k + j*v reordered as in pass 1 and Z its unnormalised N-point DFT, the spectra of the two
// real sequences are Y_k[q] = (Z[q] + conj(Z[N-q]))/2 and Y_v[q] = (Z[q] - conj(Z[N-q]))/(2j), and with
// w = exp(-j*pi*q/(2N)) * Y[q]:  C[q] = alpha[q]*Re(w),  C[N-q] = -alpha[N-q]*Im(w)  (alpha of Eq. 7).
// ---------------------------------------------------------------------------
// (P, Q) = (Z[q], Z[N-q]), t = exp(-j*pi*q/(2N)).  lo = (P_k[q], P_v[q]), hi = (P_k[N-q], P_v[N-q]).
__device__ __forceinline__ void power_of_pair(float2 P, float2 Q, float2 t, int q, float invN, float2 &lo, float2 &hi) {
  if (q == 0) {
    lo = make_float2(P.x * P.x * invN, P.y * P.y * invN);
    hi = lo;
    return;
  }
  const float2 yk = make_float2(0.5f * (P.x + Q.x), 0.5f * (P.y - Q.y));
  const float2 yv = make_float2(0.5f * (P.y + Q.y), 0.5f * (Q.x - P.x));
  const float2 wk = cmul(yk, t), wv = cmul(yv, t);
  const float a2 = 2.f * invN;
  lo = make_float2(a2 * wk.x * wk.x, a2 * wv.x * wv.x);
  hi = make_float2(a2 * wk.y * wk.y, a2 * wv.y * wv.y);
}

// Power-of-two N: pass 2 without the way back.  grid (N1/2 + 1, NY); block y works through the column
// slices y, y + NY, ... of the group and writes its sums over them to partial[y][q].
__global__ void __launch_bounds__(kThreads)
k_pass2_power(FftPlan plan, int N1, int ncol_ws, int cs2_log2, const float2 *__restrict__ ws,
              const float2 *__restrict__ master, int master_len, float2 *__restrict__ partial) {
  extern __shared__ float2 smem[];
  const int N2 = plan.len, cs2 = 1 << cs2_log2;
  const int N = N1 * N2;
  const int tid = threadIdx.x;
  const int k1a = blockIdx.x, k1b = (N1 - k1a) % N1;
  const int halves = (k1b != k1a) ? 2 : 1;
  const int ncolT_log2 = cs2_log2 + (halves - 1);
  const int ncolT = 1 << ncolT_log2;

  float2 *S = smem;                                    // [N2][2*cs2] at most
  float2 *tw = S + (size_t)N2 * 2 * cs2;               // [N2]
  float2 *twN = tw + N2;                               // [2][N2]
  unsigned short *rev = reinterpret_cast<unsigned short *>(twN + 2 * N2);   // [N2]
  unsigned short *pos_of = rev + N2;                                       // [N2]
  float2 *acc = reinterpret_cast<float2 *>(pos_of + N2);                   // [N2][2]: (P_k, P_v) of row (pos, half)

  const int mstepN = master_len / N;
  for (int i = tid; i < N2; i += kThreads) {
    tw[i] = master[(size_t)i * (master_len / N2)];
    twN[i] = master[(size_t)(((long long)i * k1a) % N) * mstepN];
    twN[N2 + i] = master[(size_t)(((long long)i * k1b) % N) * mstepN];
    const int k = digit_rev(plan, i);
    rev[i] = (unsigned short)k;
    pos_of[k] = (unsigned short)i;
    acc[2 * i] = make_float2(0.f, 0.f);
    acc[2 * i + 1] = make_float2(0.f, 0.f);
  }
  __syncthreads();

  const int tstep = master_len / (4 * N);
  const float invN = 1.f / (float)N;
  for (int sl = blockIdx.y; sl < ncol_ws / cs2; sl += gridDim.y) {
    const int gc0 = sl * cs2;
    for (int w = tid; w < N2 * ncolT; w += kThreads) {
      const int n2 = w >> ncolT_log2, col = w & (ncolT - 1);
      const int hf = col >> cs2_log2, c = col & (cs2 - 1);
      const int k1 = hf ? k1b : k1a;
      S[w] = cmul(ws[((size_t)k1 * N2 + n2) * ncol_ws + gc0 + c], twN[hf * N2 + n2]);
    }
    __syncthreads();
    fft_forward_tile(plan, S, ncolT_log2, tw, tid, kThreads);
    // every pair {q, N-q} is owned by the thread that meets the smaller bin; each location of S receives
    // the contribution of its own bin
    for (int w = tid; w < N2 * ncolT; w += kThreads) {
      const int pos = w >> ncolT_log2, col = w & (ncolT - 1);
      const int hf = col >> cs2_log2, c = col & (cs2 - 1);
      const int k1 = hf ? k1b : k1a;
      const int q = k1 + N1 * (int)rev[pos];
      const int qp = (N - q) % N;
      if (q > qp) continue;
      const int k1p = qp % N1, k2p = qp / N1;
      const int hfp = (k1p == k1) ? hf : 1 - hf;
      const int wp = ((int)pos_of[k2p] << ncolT_log2) + (hfp << cs2_log2) + c;
      float2 lo, hi;
      power_of_pair(S[w], S[wp], master[(size_t)q * tstep], q, invN, lo, hi);
      S[w] = lo;
      if (qp != q) S[wp] = hi;
    }
    __syncthreads();
    for (int r = tid; r < N2 * halves; r += kThreads) {      // row r = (pos, half): sum its cs2 columns in order
      const int pos = r / halves, hf = r - pos * halves;
      const float2 *row = S + ((size_t)pos << ncolT_log2) + (hf << cs2_log2);
      float2 a = acc[2 * pos + hf];
      for (int c = 0; c < cs2; ++c) { a.x += row[c].x; a.y += row[c].y; }
      acc[2 * pos + hf] = a;
    }
    __syncthreads();
  }
  for (int r = tid; r < N2 * halves; r += kThreads) {
    const int pos = r / halves, hf = r - pos * halves;
    const int q = (hf ? k1b : k1a) + N1 * (int)rev[pos];
    partial[(size_t)blockIdx.y * N + q] = acc[2 * pos + hf];
  }
}

// Other N (chirp path): from the N-point spectrum spec[q][col].  grid (N/2 + 1): block q sums the pair
// {q, N-q} over all columns of the group and writes partial[q], partial[N-q].
__global__ void __launch_bounds__(kThreads)
k_spec_power(const float2 *__restrict__ spec, int ncol, int N, float2 *__restrict__ partial) {
  const int q = blockIdx.x, qp = (N - q) % N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float s, c;
  sincospif(-__fdiv_rn((float)q, (float)(2 * N)), &s, &c);
  const float2 t = make_float2(c, s);
  const float invN = 1.f / (float)N;
  float a[4] = {0.f, 0.f, 0.f, 0.f};
  for (int col = tid; col < ncol; col += kThreads) {
    float2 lo, hi;
    power_of_pair(spec[(size_t)q * ncol + col], spec[(size_t)qp * ncol + col], t, q, invN, lo, hi);
    a[0] += lo.x; a[1] += lo.y; a[2] += hi.x; a[3] += hi.y;
  }
  __shared__ float red[4][kThreads / 32];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[i] = warp_sum(a[i]);
    if (lane == 0) red[i][warp] = a[i];
  }
  __syncthreads();
  if (tid == 0) {
    float r[4] = {0.f, 0.f, 0.f, 0.f};
    for (int w = 0; w < kThreads / 32; ++w)
      for (int i = 0; i < 4; ++i) r[i] += red[i][w];
    partial[q] = make_float2(r[0], r[1]);
    if (qp != q) partial[qp] = make_float2(r[2], r[3]);
  }
}

// spectrum[m] (+)= sum over y of partial[y][m], in fp64 and in a fixed order.
__global__ void k_power_accumulate(const float2 *__restrict__ partial, int ny, int N, double *__restrict__ spectrum,
                                   int first) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= N) return;
  double a = first ? 0.0 : spectrum[2 * m], b = first ? 0.0 : spectrum[2 * m + 1];
  for (int y = 0; y < ny; ++y) {
    const float2 p = partial[(size_t)y * N + m];
    a += (double)p.x;
    b += (double)p.y;
  }
  spectrum[2 * m] = a;
  spectrum[2 * m + 1] = b;
}

__global__ void k_zero_energy(double *energy) {
  if (threadIdx.x < 4) energy[threadIdx.x] = 0.0;
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
inline int ilog2(int x) { int b = 0; while ((1 << b) < x) ++b; return b; }
inline bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct SeqPlan {
  bool bluestein;
  bool fast;                 // specialised kernels (power-of-two N in [1024, 65536])
  int N, Nfft, N1, N2;
  int cs, cs2;               // columns per tile in pass 1/3 and pass 2
};

// Factors and tile widths of the generic kernels for the transform length s.Nfft.
void finish_plan(SeqPlan &s) {
  const int bits = ilog2(s.Nfft);
  int b1 = bits / 2;
  if (b1 > 7 && !s.fast) b1 = 7;
  s.cs = 64;
  // 131072 points: 256 x 512 with 32-column tiles in passes 1 and 3 beats 128 x 1024, whose pass 2 has
  // room for only 4 columns per block (measured on the chirp path: 461 against 488 ms per step)
  if (bits == 17) { b1 = 8; s.cs = 32; }
  // 8192 points on the specialised kernels: 128 x 64 keeps every pass at 256-thread blocks (2 % over 64 x 128)
  if (s.fast && bits == 13) b1 = 7;
  s.N1 = 1 << b1;
  s.N2 = s.Nfft / s.N1;
  int cs2 = 4096 / s.N2;      // 2*N2*cs2*8 bytes = 64 KiB
  if (cs2 > 64) cs2 = 64;
  if (cs2 < 4) cs2 = 4;
  s.cs2 = cs2;
}

SeqPlan plan_sequence(int N, bool allow_fast = true) {
  SeqPlan s;
  s.N = N;
  s.bluestein = !(is_pow2(N) && N >= 16);
  if (s.bluestein) {
    int M = 64;
    while (M < 2 * N - 1) M <<= 1;
    s.Nfft = M;
  } else {
    s.Nfft = N;
  }
  s.fast = allow_fast && !s.bluestein && N >= 1024 && N <= 65536;
  finish_plan(s);
  return s;
}

// Shape of a chirp transform on the specialised kernels: M = N1 * N2 with N1 = a * r1b (first-stage radix a of
// passes 1 and 3, then radix r1b) and N2 = 16 * r2b, or 2 * 16 * r2b when pass 2 takes its rows in two halves (dbl).
// Powers of two 1024..131072 have a = 16; 2^k * {5, 3, 7} have a = 10, 12, 14 with r1b = 8 or 16.  a == 0: no such
// shape.
// Channel pairs per block of passes 1 and 3 on the chirp path: with a radix-16 second stage and rows of 128 points
// or more, 16 pairs (256-thread blocks, two or three per SM) instead of 32 (512 threads, one per SM): measured
// 10..14 % on transforms of 57344..98304 points, 2 % at 28672, while 224 x 64 loses 4 % that way.
constexpr int chirp_cpw(int r1b, int r2b, bool dbl) { return (r1b == 16 && (r2b >= 8 || dbl)) ? 16 : 32; }

struct ChirpShape {
  int a, r1b, r2b;
  bool dbl;
  int n1() const { return a * r1b; }
  int n2() const { return (dbl ? 32 : 16) * r2b; }
};

inline ChirpShape chirp_shape(int M) {
  ChirpShape c{0, 0, 0, false};
  if (M == 131072) return ChirpShape{16, 16, 16, true};          // 256 x 512
  if (is_pow2(M)) {
    if (M < 1024 || M > 65536) return c;
    const int bits = ilog2(M), b1 = bits / 2;
    return ChirpShape{16, (1 << b1) / 16, (M >> b1) / 16, false};
  }
  const int a = (M % 5 == 0) ? 10 : (M % 3 == 0) ? 12 : (M % 7 == 0) ? 14 : 0;
  if (a == 0 || M % (16 * a) != 0) return c;
  // a = 10 and 12 with rows of 128 or 256 points run faster on a radix-8 second stage (80 or 96 x N2) than on
  // 160 or 192 x N2/2: measured 3..10 % on the whole chirp path; a = 14 loses 8 % that way, and rows of 512 points
  // (two halves per row in pass 2) lose 14 % against 160 or 192 x 256
  const int n2w = M / (8 * a);
  if (a != 14 && (n2w == 128 || n2w == 256)) return ChirpShape{a, 8, n2w / 16, false};
  const int n2 = M / (16 * a);
  if (!is_pow2(n2) || n2 < 32 || n2 > 512) return c;
  return n2 == 512 ? ChirpShape{a, 16, 16, true} : ChirpShape{a, 16, n2 / 16, false};
}

// Smallest transform length >= need the specialised kernels take (0 if none up to 131072).
inline int chirp_length(long long need) {
  int best = 0;
  for (int M = 1024; M <= 131072; M <<= 1)
    if (M >= need) { best = M; break; }
  for (int n1 = 160; n1 <= 224; n1 += 32)
    for (int n2 = 32; n2 <= 512; n2 <<= 1) {
      const int M = n1 * n2;
      if (M >= need && (best == 0 || M < best)) best = M;
    }
  return best;
}

struct ScoreLayout {
  size_t off_ws, off_spec, off_hhat, off_hcol, off_part_tot, off_part_hi, total;
  size_t part_tot_bytes, part_hi_bytes;   // one copy; the specialised path keeps two and alternates (step parity)
  size_t ws_buf_bytes;       // one group buffer; the fast path keeps two and alternates
  int heads_per_group;
  int sub_cols;              // chirp path: columns of one head transformed together (head_dim = all of them)
  int chirp_streams;         // chirp path: internal streams the head groups alternate over (1 = the caller's stream)
  size_t spec_buf_bytes;     // chirp path: one group's N-point spectrum; one copy per stream
  size_t layer_bytes;        // intermediates of all heads of the sequence together
};

// Workspace carve-up for one sequence plan (all sequences share the regions; the
// query takes the maximum over the sequences of the view).
ScoreLayout layout_for(const fc_handle *h, const SeqPlan &sp, int num_heads, int head_dim) {
  ScoreLayout L;
  const size_t per_head = (size_t)sp.Nfft * head_dim * sizeof(float2);
  L.layer_bytes = per_head * (size_t)num_heads;
  int hg = (int)(h->group_bytes / per_head);
  if (hg < 1) hg = 1;
  if (hg > num_heads) hg = num_heads;
  int groups = (num_heads + hg - 1) / hg;
  // Chirp transforms on the specialised kernels also alternate their head groups over the internal streams (two
  // kernels in flight fill the GPU better; measured 20-25 % on 2500..15000 tokens and still 8 % where the two
  // groups' intermediates no longer fit the L2 together).
  const bool chirp_multi = sp.bluestein && !h->generic_only && h->aux[0] != nullptr && sp.Nfft >= 1024 &&
                           sp.Nfft <= 131072 && num_heads >= h->num_aux && h->num_aux > 1;
  // Power-of-two path, all heads fit one group: they stay one group (fuller launches) and consecutive calls alternate
  // over the internal streams, where calls overlap (fc_set_score_overlap: 28 layers x 4 heads of 8192 tokens 1.31 ->
  // 1.11 ms) or the whole layer is tiny (8 MiB: 44 -> 31 us per call at 4 heads of 1024 tokens); otherwise a call
  // that has to finish before it returns is faster with its heads on both streams (49 against 56 us per layer).
  const int hg_alloc = hg;                                     // the workspace does not depend on the mode
  const bool one_group = sp.fast && groups == 1 && (h->score_overlap || L.layer_bytes <= ((size_t)8 << 20));
  if ((sp.fast || chirp_multi) && groups < h->num_aux && num_heads >= h->num_aux && !one_group)
    groups = h->num_aux;                                       // keep every internal stream busy
  hg = (num_heads + groups - 1) / groups;                      // balanced groups
  L.heads_per_group = hg;
  L.chirp_streams = chirp_multi ? h->num_aux : 1;
  // Chirp path, one head per group: the head is split into column groups only when its intermediates
  // pass four times the budget.  Narrower tiles cost time (measured: +2 % at 64 columns, +8 % at 32 for
  // 131072-point transforms) and the generic kernels do not wait on DRAM, so below that the split
  // would only save workspace.
  int sub = head_dim;
  const size_t split_above = h->group_bytes > ((size_t)1 << 60) ? h->group_bytes : 4 * h->group_bytes;
  if (sp.bluestein && hg == 1) {
    // specialised kernels: the intermediates of the groups in flight (one per internal stream) should stay in the
    // cache, so a head is halved down to 64 columns while they exceed three times the budget (measured on eight
    // ragged sequences of 7k..54k tokens: 1.6 % of the step; the length is the full form's, the band form's is shorter)
    const int Mf = h->generic_only ? 0 : chirp_length(2LL * sp.N - 1);
    if (Mf != 0 && Mf <= sp.Nfft)
      while (sub % 128 == 0 && (size_t)(chirp_multi ? h->num_aux : 1) * Mf * sub * sizeof(float2) > 3 * h->group_bytes)
        sub /= 2;
    while (sub % 64 == 0 && (size_t)sp.Nfft * sub * sizeof(float2) > split_above) sub /= 2;
  }
  L.sub_cols = sub;
  L.ws_buf_bytes = align_up((size_t)sp.Nfft * sub * (sp.fast ? hg_alloc : hg) * sizeof(float2), 256);
  size_t off = 0;
  L.off_ws = off;       off += L.ws_buf_bytes * (sp.fast ? h->num_aux : L.chirp_streams);
  L.spec_buf_bytes = sp.bluestein ? align_up((size_t)sp.N * sub * hg * sizeof(float2), 256) : 0;
  L.off_spec = off;     off += L.spec_buf_bytes * L.chirp_streams;
  L.off_hhat = off;     off += sp.bluestein ? align_up((size_t)sp.Nfft * sizeof(float2), 256) : 0;
  L.off_hcol = off;     off += sp.bluestein ? align_up((size_t)sp.Nfft * 8 * sizeof(float2), 256) : 0;
  const size_t slices = (size_t)num_heads * head_dim / 32;   // finest slicing any kernel variant uses
  L.part_tot_bytes = align_up(slices * sp.N2 * 2 * sizeof(double), 256);
  L.part_hi_bytes = align_up((size_t)num_heads * (head_dim / sub) * sp.N2 * 2 * sizeof(double), 256);
  L.off_part_tot = off; off += L.part_tot_bytes * (sp.fast ? 2 : 1);
  L.off_part_hi = off;  off += L.part_hi_bytes * (sp.fast ? 2 : 1);
  L.total = off;
  return L;
}

// The specialised path keeps each internal stream's intermediate buffer in the persisting part of L2.
// Not where the intermediates of all heads of the sequence are small against the cache (48 MiB: they stay
// resident anyway and the set-aside only takes cache from the rows and scores; measured -2.5 % at 4 heads of 8192
// tokens with the window, +1.6 % and +4 % at 2 and 4 heads of 32768, no difference at 64 MiB).
bool window_fits(const fc_handle *h, const ScoreLayout &L) {
  return h->l2_persist && L.layer_bytes > ((size_t)48 << 20) && L.ws_buf_bytes <= h->window_max &&
         L.ws_buf_bytes * (size_t)h->num_aux <= h->persist_max;
}

// The persisting part of L2 is a limit of the whole context, shared by the handles of a device (fc_persist_acquire):
// held while calls contain a sequence for the specialised path, let go when a call has none (the generic kernels
// lose about a tenth of their speed to a set-aside they do not use).  Decided once per call; left as it is while
// `st` is being captured into a graph, where device-wide settings cannot change.
void claim_persisting_l2(fc_handle *h, const fc_kv_view *kv, cudaStream_t st) {
  if (!h->l2_persist || h->generic_only) return;
  bool claim = false;
  for (int b = 0; b < kv->batch && !claim; ++b) {
    const int N = kv->cu_seqlens[b + 1] - kv->cu_seqlens[b];
    if (N == 0) continue;
    const SeqPlan sp = plan_sequence(N);
    if (!sp.fast) continue;
    claim = window_fits(h, layout_for(h, sp, kv->num_heads, kv->head_dim));
  }
  if (claim == (h->persist_on != 0)) return;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); return; }
  if (cap != cudaStreamCaptureStatusNone) return;
  if (claim) {
    if (!fc_persist_acquire(h)) h->l2_persist = 0;      // not available here: never try again
  } else {
    fc_persist_release(h);
  }
}

fc_status validate_view(const fc_handle *h, const fc_kv_view *kv) {
  if (!h || !kv || !kv->k || !kv->v || !kv->cu_seqlens) return FC_ERR_INVALID_ARG;
  if (kv->num_heads <= 0 || kv->head_dim <= 0 || kv->batch < 0) return FC_ERR_INVALID_ARG;
  if (kv->dtype != FC_F32 && kv->dtype != FC_F16 && kv->dtype != FC_BF16) return FC_ERR_UNSUPPORTED;
  if (kv->head_dim % 64 != 0) return FC_ERR_UNSUPPORTED;
  const size_t es = kv->dtype == FC_F32 ? 4 : 2;
  if (kv->cu_seqlens[0] != 0) return FC_ERR_INVALID_ARG;
  for (int b = 0; b < kv->batch; ++b) {
    const long long n = (long long)kv->cu_seqlens[b + 1] - kv->cu_seqlens[b];
    if (n < 0) return FC_ERR_INVALID_ARG;
    if (n > h->max_seqlen) return FC_ERR_UNSUPPORTED;
    if (n > 65536 && !is_pow2((int)n)) return FC_ERR_UNSUPPORTED;
  }
  if (kv->stride_token < (long long)kv->head_dim || kv->stride_head < (long long)kv->head_dim)
    return FC_ERR_INVALID_ARG;
  if (((uintptr_t)kv->k & 15) || ((uintptr_t)kv->v & 15)) return FC_ERR_INVALID_ARG;
  if ((kv->stride_token * es) % 16 || (kv->stride_head * es) % 16) return FC_ERR_INVALID_ARG;
  return FC_OK;
}

// Function attributes are set once per kernel and device (and again only if a launch needs more shared
// memory than the last time), not before every launch.
template <class Kern>
fc_status set_smem(Kern kern, size_t bytes) {
  static std::mutex mu;
  static std::unordered_map<unsigned long long, size_t> done;     // (device, kernel) -> bytes already allowed
  int dev = 0;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  const unsigned long long key = (unsigned long long)reinterpret_cast<uintptr_t>(reinterpret_cast<const void *>(kern)) ^
                                 ((unsigned long long)dev << 56);
  std::lock_guard<std::mutex> lock(mu);
  auto it = done.find(key);
  if (it != done.end() && it->second >= bytes) return FC_OK;
  if (bytes > 48 * 1024) FC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
  // as much of the L1/shared array as shared memory as the device offers: these kernels do not rely on L1
  if (it == done.end())
    FC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
  done[key] = bytes;
  return FC_OK;
}

size_t smem_pass13(const SeqPlan &sp, int cs) {
  return (size_t)sp.N1 * cs * sizeof(float2) + sp.N1 * sizeof(float2) + sp.N1 * sizeof(int) + 2 * sp.N1 * sizeof(float);
}
size_t smem_pass2(const SeqPlan &sp, int cs2, int halves = 2) {
  return (size_t)sp.N2 * halves * cs2 * sizeof(float2) + 3 * (size_t)sp.N2 * sizeof(float2) + 2 * (size_t)sp.N2 * sizeof(unsigned short);
}

template <class Loader>
fc_status launch_pass1(fc_handle *h, cudaStream_t st, const Loader &ld, const SeqPlan &sp, int ncol_ws, int cs,
                       float2 *ws, double *partial) {
  const FftPlan p1 = make_plan(sp.N1);
  const size_t sm = smem_pass13(sp, cs);
  fc_status s = set_smem(k_pass1<Loader>, sm);
  if (s != FC_OK) return s;
  dim3 grid(sp.N2, ncol_ws / cs);
  ProfScope ps(h, FC_K_PASS1, st);
  k_pass1<Loader><<<grid, kThreads, sm, st>>>(ld, p1, sp.N2, ncol_ws, ilog2(cs), ws, h->master, h->master_len, partial);
  return fc_after_launch(h);
}

template <int MID>
fc_status launch_pass2(fc_handle *h, cudaStream_t st, const SeqPlan &sp, int ncol_ws, int cs2, float2 *ws,
                       int omega, float2 *hhat, float scale) {
  const FftPlan p2 = make_plan(sp.N2);
  const size_t sm = smem_pass2(sp, cs2, MID == MID_DCT ? 2 : 1);
  fc_status s = set_smem(k_pass2<MID>, sm);
  if (s != FC_OK) return s;
  dim3 grid(MID == MID_DCT ? sp.N1 / 2 + 1 : sp.N1, ncol_ws / cs2);
  ProfScope ps(h, FC_K_PASS2, st);
  k_pass2<MID><<<grid, kThreads, sm, st>>>(p2, sp.N1, ncol_ws, ilog2(cs2), ws, h->master, h->master_len, omega, hhat, scale);
  return fc_after_launch(h);
}

// The three specialised launches for one head group of a power-of-two sequence.
// Channel pairs per block of passes 1 and 3 on the power-of-two path for a first factor n1.
constexpr int fast_cpw(int n1, int cpw) { return n1 == 256 ? 16 : cpw; }

// CPW: channel pairs per block in passes 1 and 3; CP: channel pairs per half tile in pass 2.
template <typename T, int R1B, int R2B, int CPW, int CP>
fc_status launch_fast_impl(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, const T *kp, const T *vp,
                           const SeqPlan &sp, int h0, int hg, int omega, float2 *ws, double *ptot,
                           double *phi, float *scores, long long total_tokens, const double *part_tot,
                           const double *part_hi, double *energy_b) {
  constexpr int N1 = 16 * R1B, N2 = 16 * R2B;
  const int d = kv->head_dim, ncol_ws = hg * d;
  const size_t sm1 = (size_t)N1 * CPW * sizeof(float4) + N1 * sizeof(float2);
  const size_t sm2 = (size_t)2 * N2 * CP * sizeof(float4) + (5 * N2 + 16) * sizeof(float2);
  fc_status s;
  if ((s = set_smem(fast::k_p1<T, R1B, CPW>, sm1)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS1, st);
    fast::k_p1<T, R1B, CPW><<<dim3(N2, ncol_ws / (2 * CPW)), CPW * R1B, sm1, st>>>(
        kp, vp, kv->stride_token, kv->stride_head, h0, d, sp.N, N2, ncol_ws, ws, h->master, h->master_len, ptot);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  if ((s = set_smem(fast::k_p2<R2B, CP>, sm2)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS2, st);
    fast::k_p2<R2B, CP><<<dim3(N1 / 2, ncol_ws / (2 * CP)), 2 * CP * R2B, sm2, st>>>(
        N1, ncol_ws, ws, h->master, h->master_len, omega);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  if ((s = set_smem(fast::k_p3<R1B, CPW>, sm1)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS3, st);
    const float inv = (float)(1.0 / ((double)sp.N * (double)sp.N * (double)d));
    const int H = kv->num_heads;
    fast::k_p3<R1B, CPW><<<dim3(N2, hg), CPW * R1B, sm1, st>>>(
        sp.N, N2, ncol_ws, ws, h->master, h->master_len, scores, h0, d, total_tokens, inv, phi,
        h->done_counter + (h->step & 1u), (unsigned)(N2 * H), part_tot, N2 * (H * d / (2 * CPW)), part_hi, N2 * H, energy_b);
  }
  return fc_after_launch(h);
}

template <typename T, int CPW, int CP>
fc_status launch_fast_tuned(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, const T *kp, const T *vp,
                            const SeqPlan &sp, int h0, int hg, int omega, float2 *ws, double *ptot, double *phi,
                            float *scores, long long total_tokens, const double *part_tot,
                            const double *part_hi, double *energy_b) {
  // Every pass runs 256-thread blocks, the measured optimum: CPWV channel pairs per block in passes 1 and 3 and CPV
  // per half tile in pass 2 follow from the factors (CPW and CP are the widths for 128 x 256).
#define FC_FAST_CASE(A, B, CPWV, CPV)                                                                     \
  if (sp.N1 == 16 * A && sp.N2 == 16 * B)                                                                 \
    return launch_fast_impl<T, A, B, CPWV, CPV>(h, st, kv, kp, vp, sp, h0, hg, omega, ws, ptot, phi, scores, \
                                                total_tokens, part_tot, part_hi, energy_b);
  FC_FAST_CASE(2, 2, CPW, CP) FC_FAST_CASE(2, 4, CPW, CP) FC_FAST_CASE(4, 4, CPW, CP) FC_FAST_CASE(4, 8, CPW, CP)
  FC_FAST_CASE(8, 4, CPW, 4 * CP)                 // 8192 = 128 x 64
  FC_FAST_CASE(8, 8, CPW, 2 * CP)                 // 16384 = 128 x 128
  FC_FAST_CASE(8, 16, CPW, CP)                    // 32768 = 128 x 256
  FC_FAST_CASE(16, 16, fast_cpw(256, CPW), CP)    // 65536 = 256 x 256
#undef FC_FAST_CASE
  return FC_ERR_INTERNAL;
}

template <typename T>
fc_status launch_fast(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, const T *kp, const T *vp,
                      const SeqPlan &sp, int h0, int hg, int omega, float2 *ws, double *ptot, double *phi,
                      float *scores, long long total_tokens, const double *part_tot, const double *part_hi,
                      double *energy_b) {
#define FC_TUNE_CASE(W, C)                                                                              \
  if (h->tune_cpw == W && h->tune_cp == C)                                                              \
    return launch_fast_tuned<T, W, C>(h, st, kv, kp, vp, sp, h0, hg, omega, ws, ptot, phi, scores,       \
                                      total_tokens, part_tot, part_hi, energy_b);
  FC_TUNE_CASE(32, 8)
#undef FC_TUNE_CASE
  return FC_ERR_INTERNAL;
}

// The chirp path on the specialised kernels: two circular convolutions with the chirp kernel, each
// pass 1 -> pass 2 (multiply by the kernel's spectrum) -> pass 3, on one stream.  Tile widths fixed.
// DOUBLE: rows of 2 * 16 * R2B points, pass 2 joins two half-length transforms per row.
// hout != nullptr: only the spectrum of the convolution kernel itself is computed (pass 1 with the kernel in column
// 0 of a 64-column tile, the forward half of pass 2) and written to hout[0 .. M).
template <typename T, int A, int R1B, int R2B, bool DOUBLE>
fc_status launch_chirp_impl(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, const T *kp, const T *vp, int Nseq,
                            int h0, int hg, int omega, float2 *ws, float2 *spec, const float2 *hhat, double *ptot,
                            double *phi, float *scores, long long total_tokens, int dcols, int accumulate, int band,
                            float2 *hout, const float2 *ctab) {
  constexpr int CPW = chirp_cpw(R1B, R2B, DOUBLE), CP = 8, N1 = A * R1B, N2 = (DOUBLE ? 32 : 16) * R2B;
  constexpr int MIDV = DOUBLE ? fast::MID_CONV2 : fast::MID_CONV;
  const size_t sm1 = (size_t)N1 * CPW * sizeof(float4) + N1 * sizeof(float2);
  const size_t sm2 = (size_t)2 * (16 * R2B) * CP * sizeof(float4) + (7 * (16 * R2B) + 16) * sizeof(float2);
  // band form's last pass, 16-bit inputs: staging slots for the K/V rows it reads again
  const size_t sm3b = sm1 + (sizeof(T) == 2 ? (size_t)2 * A * CPW * R1B * sizeof(unsigned) : 0);
  fc_status s;
  if ((s = set_smem(fast::k_p2<R2B, CP, MIDV>, sm2)) != FC_OK) return s;
  if (hout != nullptr) {
    if ((s = set_smem(fast::k_p1<float, R1B, CPW, fast::LD_KERNEL, A>, sm1)) != FC_OK) return s;
    {
      ProfScope ps(h, FC_K_PASS1, st);
      fast::k_p1<float, R1B, CPW, fast::LD_KERNEL, A><<<dim3(N2, 1), CPW * R1B, sm1, st>>>(
          nullptr, nullptr, 0, 0, 0, 2 * CPW, Nseq, N2, 2 * CPW, ws, h->master, h->master_len, nullptr, nullptr, band);
    }
    if ((s = fc_after_launch(h)) != FC_OK) return s;
    {
      ProfScope ps(h, FC_K_PASS2, st);
      fast::k_p2<R2B, CP, MIDV><<<dim3(DOUBLE ? N1 : N1 / 2, 1), 2 * CP * R2B, sm2, st>>>(
          N1, 2 * CPW, ws, h->master, h->master_len, 0, nullptr, 1.f, 0, hout);
    }
    return fc_after_launch(h);
  }
  // dcols: columns of a head in this launch (head_dim, or a column group of one head: kp/vp point at its
  // first channel and hg is 1)
  const int d = kv->head_dim, ncol = hg * dcols;
  const float invM = 1.f / (float)(N1 * N2);
  const dim3 g1(N2, ncol / (2 * CPW)), g2(DOUBLE ? N1 : N1 / 2, ncol / (2 * CP)), g3(N2, hg);
  if ((s = set_smem(fast::k_p1<T, R1B, CPW, fast::LD_CHIRP, A>, sm1)) != FC_OK) return s;
  if ((s = set_smem(fast::k_p3<R1B, CPW, fast::OUT_SPEC, float, A>, sm1)) != FC_OK) return s;
  if (band >= 0) {
    if ((s = set_smem(fast::k_p1<float, R1B, CPW, fast::LD_BAND, A>, sm1)) != FC_OK) return s;
    if ((s = set_smem(fast::k_p3<R1B, CPW, fast::OUT_SCORE_BAND, T, A>, sm3b)) != FC_OK) return s;
  } else {
    if ((s = set_smem(fast::k_p1<float, R1B, CPW, fast::LD_FILTER, A>, sm1)) != FC_OK) return s;
    if ((s = set_smem(fast::k_p3<R1B, CPW, fast::OUT_SCORE_CHIRP, float, A>, sm1)) != FC_OK) return s;
  }
  {
    ProfScope ps(h, FC_K_PASS1, st);
    fast::k_p1<T, R1B, CPW, fast::LD_CHIRP, A><<<g1, CPW * R1B, sm1, st>>>(
        kp, vp, kv->stride_token, kv->stride_head, h0, dcols, Nseq, N2, ncol, ws, h->master, h->master_len, ptot,
        nullptr, 0, ctab);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS2, st);
    fast::k_p2<R2B, CP, MIDV><<<g2, 2 * CP * R2B, sm2, st>>>(N1, ncol, ws, h->master, h->master_len, 0, hhat, invM);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS3, st);
    fast::k_p3<R1B, CPW, fast::OUT_SPEC, float, A><<<g3, CPW * R1B, sm1, st>>>(
        Nseq, N2, ncol, ws, h->master, h->master_len, nullptr, h0, dcols, 0, 0.f, nullptr, nullptr, 0u, nullptr, 0, nullptr, 0,
        nullptr, spec, 0.f, 0, band, nullptr, nullptr, 0, 0, ctab);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS1, st);
    if (band >= 0)
      fast::k_p1<float, R1B, CPW, fast::LD_BAND, A><<<g1, CPW * R1B, sm1, st>>>(
          nullptr, nullptr, 0, 0, 0, ncol, Nseq, N2, ncol, ws, h->master, h->master_len, nullptr, spec, band, ctab);
    else
      fast::k_p1<float, R1B, CPW, fast::LD_FILTER, A><<<g1, CPW * R1B, sm1, st>>>(
          nullptr, nullptr, 0, 0, 0, ncol, Nseq, N2, ncol, ws, h->master, h->master_len, nullptr, spec, omega, ctab);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  {
    // band form: the second convolution's kernel is the first one's read backwards, whose spectrum is hhat read
    // backwards
    ProfScope ps(h, FC_K_PASS2, st);
    fast::k_p2<R2B, CP, MIDV><<<g2, 2 * CP * R2B, sm2, st>>>(N1, ncol, ws, h->master, h->master_len, 0, hhat, invM,
                                                             band >= 0 ? 1 : 0);
  }
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  {
    ProfScope ps(h, FC_K_PASS3, st);
    if (band >= 0) {
      fast::k_p3<R1B, CPW, fast::OUT_SCORE_BAND, T, A><<<g3, CPW * R1B, sm3b, st>>>(
          Nseq, N2, ncol, ws, h->master, h->master_len, scores, h0, dcols, total_tokens, (float)(1.0 / (double)d), phi,
          nullptr, 0u, nullptr, 0, nullptr, 0, nullptr, nullptr, (float)d, accumulate, band, kp, vp, kv->stride_token,
          kv->stride_head, ctab);
    } else {
      const float inv = (float)(1.0 / ((double)Nseq * (double)Nseq * (double)d));
      fast::k_p3<R1B, CPW, fast::OUT_SCORE_CHIRP, float, A><<<g3, CPW * R1B, sm1, st>>>(
          Nseq, N2, ncol, ws, h->master, h->master_len, scores, h0, dcols, total_tokens, inv, phi, nullptr, 0u, nullptr, 0,
          nullptr, 0, nullptr, nullptr, (float)d, accumulate, -1, nullptr, nullptr, 0, 0, ctab);
    }
  }
  return fc_after_launch(h);
}

template <typename T>
fc_status launch_chirp(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, const T *kp, const T *vp, int Nseq, int M,
                       int h0, int hg, int omega, float2 *ws, float2 *spec, const float2 *hhat, double *ptot,
                       double *phi, float *scores, long long total_tokens, int dcols, int accumulate, int band,
                       const float2 *ctab, float2 *hout = nullptr) {
  const ChirpShape c = chirp_shape(M);
#define FC_CHIRP_CASE(A, B, C, D)                                                                               \
  if (c.a == A && c.r1b == B && c.r2b == C && c.dbl == D)                                                       \
    return launch_chirp_impl<T, A, B, C, D>(h, st, kv, kp, vp, Nseq, h0, hg, omega, ws, spec, hhat, ptot, phi, \
                                            scores, total_tokens, dcols, accumulate, band, hout, ctab);
  FC_CHIRP_CASE(16, 2, 2, false) FC_CHIRP_CASE(16, 2, 4, false) FC_CHIRP_CASE(16, 4, 4, false)
  FC_CHIRP_CASE(16, 4, 8, false) FC_CHIRP_CASE(16, 8, 8, false) FC_CHIRP_CASE(16, 8, 16, false)
  FC_CHIRP_CASE(16, 16, 16, false) FC_CHIRP_CASE(16, 16, 16, true)
  // a = 14: 224 x {32 .. 512}
  FC_CHIRP_CASE(14, 16, 2, false) FC_CHIRP_CASE(14, 16, 4, false) FC_CHIRP_CASE(14, 16, 8, false)
  FC_CHIRP_CASE(14, 16, 16, false) FC_CHIRP_CASE(14, 16, 16, true)
  // a = 10, 12: {160, 192} x 32, {80, 96} x {128, 256}, {160, 192} x {256, 512}
  FC_CHIRP_CASE(10, 16, 2, false) FC_CHIRP_CASE(10, 8, 8, false) FC_CHIRP_CASE(10, 8, 16, false)
  FC_CHIRP_CASE(10, 16, 16, false) FC_CHIRP_CASE(10, 16, 16, true)
  FC_CHIRP_CASE(12, 16, 2, false) FC_CHIRP_CASE(12, 8, 8, false) FC_CHIRP_CASE(12, 8, 16, false)
  FC_CHIRP_CASE(12, 16, 16, false) FC_CHIRP_CASE(12, 16, 16, true)
#undef FC_CHIRP_CASE
  return FC_ERR_INTERNAL;
}

// Cutoff index omega of Eq. 8 for a sequence of N tokens.
inline int cutoff_index(double gamma, int N) {
  long long om = (long long)floor(gamma * (double)N);
  if (om > N - 1) om = N - 1;
  if (om < 0) om = 0;
  return (int)om;
}

// Convolution length of the chirp path.  Full form: M >= 2N - 1.  Band form: only the bins -omega .. omega of the
// spectrum are needed (the low-pass part; the score is taken against the input rows), M >= N + 2*omega + 1.  The
// specialised kernels take powers of two and 2^k * {3, 5, 7}; whichever form gives the shorter M runs, and the
// generic kernels (M = sp.Nfft, a power of two, full form) remain for what the specialised ones do not take
// (cols_ok: the column groups are multiples of 64 channels).
struct ChirpChoice {
  int band;      // omega when the band form runs, else -1
  int M;         // convolution length
  bool fast;     // specialised kernels
};

inline ChirpChoice choose_chirp(const fc_handle *h, const SeqPlan &sp, int N, int omega, bool cols_ok) {
  ChirpChoice c{-1, sp.Nfft, false};
  if (!sp.bluestein || h->generic_only || !cols_ok) return c;
  const int Mf = chirp_length(2LL * N - 1);
  if (Mf != 0 && Mf <= sp.Nfft) { c.M = Mf; c.fast = true; }
  if (h->band_form && 2LL * omega + 1 < N) {
    const int Mb = chirp_length((long long)N + 2LL * omega + 1);
    if (Mb != 0 && Mb < c.M) { c.band = omega; c.M = Mb; c.fast = true; }
  }
  return c;
}

template <typename T>
fc_status score_sequence(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, int b, double gamma,
                         float *scores, double *energy, char *wsb) {
  const int start = kv->cu_seqlens[b];
  const int N = kv->cu_seqlens[b + 1] - start;
  const long long total_tokens = kv->cu_seqlens[kv->batch];
  double *energy_b = energy + 4 * (size_t)b;
  if (N == 0) {
    k_zero_energy<<<1, 32, 0, st>>>(energy_b);
    return fc_after_launch(h);
  }
  const int d = kv->head_dim, H = kv->num_heads;
  const SeqPlan sp = plan_sequence(N, !h->generic_only);
  const ScoreLayout L = layout_for(h, sp, H, d);
  const int omega = cutoff_index(gamma, N);

  fc_status s0 = FC_OK;
  float2 *ws = reinterpret_cast<float2 *>(wsb + L.off_ws);
  float2 *spec = reinterpret_cast<float2 *>(wsb + L.off_spec);
  float2 *hhat = reinterpret_cast<float2 *>(wsb + L.off_hhat);
  float2 *hcol = reinterpret_cast<float2 *>(wsb + L.off_hcol);
  double *part_tot = reinterpret_cast<double *>(wsb + L.off_part_tot);
  double *part_hi = reinterpret_cast<double *>(wsb + L.off_part_hi);
  const bool separate_fast = sp.fast;
  if (separate_fast) {                 // consecutive steps alternate between two copies of the partial sums
    part_tot = reinterpret_cast<double *>(wsb + L.off_part_tot + (h->step & 1u) * L.part_tot_bytes);
    part_hi = reinterpret_cast<double *>(wsb + L.off_part_hi + (h->step & 1u) * L.part_hi_bytes);
  } else {
    if ((s0 = fc_flush_pending(h, st)) != FC_OK) return s0;   // this path works on the caller's stream
  }
  const T *kp = static_cast<const T *>(kv->k) + (long long)start * kv->stride_token;
  const T *vp = static_cast<const T *>(kv->v) + (long long)start * kv->stride_token;
  const FftPlan p1 = make_plan(sp.N1);
  fc_status s;

  const ChirpChoice cc = choose_chirp(h, sp, N, omega, L.sub_cols % 64 == 0);
  const int band = cc.band, Mc = cc.M;
  const bool chirp_fast = cc.fast;
  SeqPlan spc = sp;                      // plan of the convolution length, for the generic kernels
  if (is_pow2(Mc)) { spc.Nfft = Mc; finish_plan(spc); }

  const float2 *ctab = nullptr;
  if (sp.bluestein) {
    // Spectrum of the chirp kernel.  It depends on the sequence length only, so the handle keeps the last few
    // (layers of a prefill share their lengths).  While the stream is being captured the spectrum goes to the
    // workspace instead, every time: a graph must not depend on what the handle holds when it is replayed.
    bool cached = false;
    if (h->hhat_cache && !h->generic_only && sp.Nfft <= h->hhat_cache_len) {
      cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
      if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusActive; }
      cached = (cap == cudaStreamCaptureStatusNone);
    }
    bool have = false;
    int slot = 0;
    const long long hkey = (long long)N + ((long long)(band + 1) << 32);
    if (cached) {
      for (int i = 0; i < FC_HHAT_SLOTS && !have; ++i)
        if (h->hhat_cache_n[i] == hkey) { have = true; slot = i; }
      if (!have) {
        // the slot taken over was last read by a sequence that has been joined to `st` since (the chirp path
        // joins the internal streams before it returns), so stream order protects it
        slot = h->hhat_cache_next;
        h->hhat_cache_next = (slot + 1) % FC_HHAT_SLOTS;
        h->hhat_cache_n[slot] = 0;                          // not valid until both launches are in the stream
      }
      hhat = h->hhat_cache + (size_t)slot * h->hhat_slot_len;
    }
    if (!have) {
      if (is_pow2(Mc)) {
        ChirpKernelLoader cl{N, Mc, band};
        if ((s = launch_pass1(h, st, cl, spc, 8, 8, hcol, nullptr)) != FC_OK) return s;
        if ((s = launch_pass2<MID_SPEC>(h, st, spc, 8, 8, hcol, 0, hhat, 1.f)) != FC_OK) return s;
      } else {
        // lengths with an odd factor: the specialised kernels transform the kernel themselves (64 columns of the
        // workspace, which no head group uses yet)
        if ((s = launch_chirp<T>(h, st, kv, nullptr, nullptr, N, Mc, 0, 1, 0, ws, nullptr, nullptr, nullptr, nullptr,
                                 nullptr, 0, 64, 0, band, nullptr, hhat)) != FC_OK) return s;
      }
      if (cached) h->hhat_cache_n[slot] = hkey;
    }
    // per-row factors of the chirp modes (2N values): behind the spectrum in its cache slot, else in the column
    // buffer of the workspace, which the spectrum's transform no longer needs
    ctab = cached ? hhat + h->hhat_cache_len : hcol;
    if (!have && chirp_fast) {
      ProfScope ps(h, FC_K_OTHER, st);
      fast::k_chirp_tables<<<(N + 255) / 256, 256, 0, st>>>(const_cast<float2 *>(ctab), N);
      if ((s = fc_after_launch(h)) != FC_OK) return s;
    }
  }

  // fc_score_layer has claimed the persisting part of L2 if any sequence of the call takes this path
  const bool want_persist = separate_fast && window_fits(h, L);
  if (want_persist && h->persist_on) {
    // keep each stream's intermediate in the persisting part of L2; everything else these streams touch
    // (the K/V rows, the scores) streams through
    for (int i = 0; i < h->num_aux; ++i) {
      const char *base = wsb + L.off_ws + (size_t)i * L.ws_buf_bytes;
      if (h->window_base[i] == base && h->window_bytes[i] == L.ws_buf_bytes) continue;
      cudaStreamAttrValue av = {};
      av.accessPolicyWindow.base_ptr = const_cast<char *>(base);
      av.accessPolicyWindow.num_bytes = L.ws_buf_bytes;
      av.accessPolicyWindow.hitRatio = 1.0f;
      av.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
      av.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
      if (cudaStreamSetAttribute(h->aux[i], cudaStreamAttributeAccessPolicyWindow, &av) != cudaSuccess) {
        cudaGetLastError();
        h->l2_persist = 0;               // not supported here: never try again
        break;
      }
      h->window_base[i] = base;
      h->window_bytes[i] = L.ws_buf_bytes;
    }
  }
  if (sp.fast) {
    const long long sig = (long long)N + ((long long)H << 20) + ((long long)d << 40);
    FC_CUDA_TRY(cudaEventRecord(h->ev_fork, st));
    for (int i = 0; i < h->num_aux; ++i) {
      FC_CUDA_TRY(cudaStreamWaitEvent(h->aux[i], h->ev_fork, 0));
      for (int o = 0; o < h->num_aux; ++o) {
        if (o == i) continue;
        // the partial sums and the block counter of this parity were last used two steps ago: the other
        // streams must be through with that step (this one is, by stream order)
        if (h->step >= 2) FC_CUDA_TRY(cudaStreamWaitEvent(h->aux[i], h->ev_done[h->step & 1u][o], 0));
        // a different shape carves the workspace differently: nothing of the previous step may be in flight
        if (h->step >= 1 && sig != h->last_sig)
          FC_CUDA_TRY(cudaStreamWaitEvent(h->aux[i], h->ev_done[(h->step - 1) & 1u][o], 0));
      }
    }
    h->last_sig = sig;
  }
  const bool chirp_fork = sp.bluestein && L.chirp_streams > 1;
  if (chirp_fork) {                     // the internal streams start after the chirp kernel's spectrum is ready
    FC_CUDA_TRY(cudaEventRecord(h->ev_fork, st));
    for (int i = 0; i < L.chirp_streams; ++i) FC_CUDA_TRY(cudaStreamWaitEvent(h->aux[i], h->ev_fork, 0));
  }
  size_t tot_slots = 0, hi_slots = 0;
  int group = 0;
  for (int h0 = 0; h0 < H; h0 += L.heads_per_group, ++group) {
    const int hg = (H - h0 < L.heads_per_group) ? H - h0 : L.heads_per_group;
    const int ncol_ws = hg * d;
    double *ptot = part_tot + 2 * tot_slots;
    double *phi = part_hi + 2 * hi_slots;
    const size_t sm3 = smem_pass13(sp, sp.cs);
    if (sp.fast) {
      const int si = (int)((group + h->step) % (unsigned)h->num_aux);   // a single group: steps alternate
      float2 *wsg = reinterpret_cast<float2 *>(wsb + L.off_ws + (size_t)si * L.ws_buf_bytes);
      if ((s = launch_fast<T>(h, h->aux[si], kv, kp, vp, sp, h0, hg, omega, wsg, ptot, phi,
                              scores + start, total_tokens, part_tot, part_hi, energy_b)) != FC_OK) return s;
    } else if (!sp.bluestein) {
      KvLoader<T, false> ld{kp, vp, kv->stride_token, kv->stride_head, h0, d, N, 0.f, 0.f};
      if ((s = launch_pass1(h, st, ld, sp, ncol_ws, sp.cs, ws, ptot)) != FC_OK) return s;
      if ((s = launch_pass2<MID_DCT>(h, st, sp, ncol_ws, sp.cs2, ws, omega, nullptr, 1.f / (float)N)) != FC_OK) return s;
      if ((s = set_smem(k_pass3<EPI_SCORE, false>, sm3)) != FC_OK) return s;
      {
        ProfScope ps(h, FC_K_PASS3, st);
        k_pass3<EPI_SCORE, false><<<dim3(sp.N2, hg), kThreads, sm3, st>>>(
            p1, sp.N2, N, ncol_ws, ilog2(sp.cs), ws, h->master, h->master_len, nullptr, scores + start, h0, d,
            total_tokens, 1.f / (float)d, phi, (float)d, 0);
      }
      if ((s = fc_after_launch(h)) != FC_OK) return s;
    } else {
      // One head may be transformed in several column groups (sub < d) so that the padded
      // length-Nfft intermediates of a group stay within the cache budget; the groups run in
      // stream order and the last pass adds their contributions to the score in that order.
      if (chirp_fast) {                         // a length and a width the specialised kernels take
        const int sub = L.sub_cols, ngr = (hg == 1) ? d / sub : 1, n2f = chirp_shape(Mc).n2();
        const ChirpShape shp = chirp_shape(Mc);
        const int tilew = 2 * chirp_cpw(shp.r1b, shp.r2b, shp.dbl);     // columns per block of passes 1 and 3
        const int ncol = (hg == 1) ? sub : ncol_ws;
        const int si = group % L.chirp_streams;                   // head groups alternate over the internal streams
        cudaStream_t sx = L.chirp_streams > 1 ? h->aux[si] : st;
        float2 *ws_s = reinterpret_cast<float2 *>(wsb + L.off_ws + (size_t)si * L.ws_buf_bytes);
        float2 *spec_s = reinterpret_cast<float2 *>(wsb + L.off_spec + (size_t)si * L.spec_buf_bytes);
        for (int cg = 0; cg < ngr; ++cg) {                        // column groups of one head, else one pass
          if ((s = launch_chirp<T>(h, sx, kv, kp + cg * sub, vp + cg * sub, N, Mc, h0, hg, omega, ws_s, spec_s, hhat,
                                   ptot + 2 * (size_t)cg * n2f * (ncol / tilew), phi + 2 * (size_t)cg * n2f * hg,
                                   scores + start, total_tokens, (hg == 1) ? sub : d, cg > 0 ? 1 : 0, band, ctab)) != FC_OK)
            return s;
        }
        tot_slots += (size_t)n2f * (ncol / tilew) * ngr;
        hi_slots += (size_t)n2f * hg * ngr;
        continue;
      }
      const float invM = 1.f / (float)sp.Nfft;
      const float inv = (float)(1.0 / ((double)N * (double)N * (double)d));
      const int sub = L.sub_cols, cs = (sub % 64 == 0) ? sp.cs : 32;
      const int ngroups = (hg == 1) ? d / sub : 1;
      const int ncol = (hg == 1) ? sub : ncol_ws;
      int cs2 = 2 * sp.cs2 > 64 ? 64 : 2 * sp.cs2;       // the convolution pass holds single rows: twice the columns fit
      while (ncol % cs2) cs2 >>= 1;
      const size_t sm3c = smem_pass13(sp, cs);
      for (int cg = 0; cg < ngroups; ++cg) {
        const int c0 = cg * sub;
        double *ptot_c = ptot + 2 * (size_t)cg * sp.N2 * (ncol / cs);
        double *phi_c = phi + 2 * (size_t)cg * sp.N2 * hg;
        const int dd = (hg == 1) ? sub : d;           // columns the loader and the last pass see per head
        KvLoader<T, true> ld{kp + c0, vp + c0, kv->stride_token, kv->stride_head, h0, dd, N, 0.f, 0.f};
        if ((s = launch_pass1(h, st, ld, sp, ncol, cs, ws, ptot_c)) != FC_OK) return s;
        if ((s = launch_pass2<MID_MULH>(h, st, sp, ncol, cs2, ws, 0, hhat, invM)) != FC_OK) return s;
        if ((s = set_smem(k_pass3<EPI_SPEC, true>, sm3c)) != FC_OK) return s;
        {
          ProfScope ps(h, FC_K_PASS3, st);
          k_pass3<EPI_SPEC, true><<<dim3(sp.N2, ncol / cs), kThreads, sm3c, st>>>(
              p1, sp.N2, N, ncol, ilog2(cs), ws, h->master, h->master_len, spec, nullptr, 0, dd, 0, 0.f, nullptr,
              0.f, 0);
        }
        if ((s = fc_after_launch(h)) != FC_OK) return s;
        FilterLoader fl{spec, ncol, N, omega};
        if ((s = launch_pass1(h, st, fl, sp, ncol, cs, ws, nullptr)) != FC_OK) return s;
        if ((s = launch_pass2<MID_MULH>(h, st, sp, ncol, cs2, ws, 0, hhat, invM)) != FC_OK) return s;
        if ((s = set_smem(k_pass3<EPI_SCORE, true>, sm3c)) != FC_OK) return s;
        {
          ProfScope ps(h, FC_K_PASS3, st);
          k_pass3<EPI_SCORE, true><<<dim3(sp.N2, hg), kThreads, sm3c, st>>>(
              p1, sp.N2, N, ncol, ilog2(cs), ws, h->master, h->master_len, nullptr, scores + start, h0, dd,
              total_tokens, inv, phi_c, (float)d, cg > 0 ? 1 : 0);
        }
        if ((s = fc_after_launch(h)) != FC_OK) return s;
      }
      tot_slots += (size_t)sp.N2 * (ncol / cs) * ngroups;
      hi_slots += (size_t)sp.N2 * hg * ngroups;
      continue;
    }
    tot_slots += (size_t)sp.N2 * (ncol_ws / (sp.fast ? 2 * fast_cpw(sp.N1, h->tune_cpw) : sp.cs));
    hi_slots += (size_t)sp.N2 * hg;
  }
  if (sp.fast) {
    for (int i = 0; i < h->num_aux; ++i) FC_CUDA_TRY(cudaEventRecord(h->ev_done[h->step & 1u][i], h->aux[i]));
    h->step++;
    h->pending_join = true;
    if (!h->score_overlap) {           // default: the caller's stream waits for this call's work right away
      if ((s = fc_flush_pending(h, st)) != FC_OK) return s;
    }
  }
  if (sp.fast) return FC_OK;          // the last pass-3 block of the sequence has written the energy sums
  if (chirp_fork) {                     // the caller's stream takes over again for the energy sums
    for (int i = 0; i < L.chirp_streams; ++i) {
      FC_CUDA_TRY(cudaEventRecord(h->ev_join[i], h->aux[i]));
      FC_CUDA_TRY(cudaStreamWaitEvent(st, h->ev_join[i], 0));
    }
  }
  {
    ProfScope ps(h, FC_K_OTHER, st);
    k_energy_finalize<<<1, 256, 0, st>>>(part_tot, (int)tot_slots, part_hi, (int)hi_slots, energy_b);
  }
  return fc_after_launch(h);
}

// Column slices of one launch of k_pass2_power that run side by side (the rest are looped over).
constexpr int kPowerNY = 16;

size_t power_partial_bytes(int N) { return align_up((size_t)kPowerNY * N * sizeof(float2), 256); }

// Power spectrum of one sequence (Eq. 11) into spectrum[2*m .. 2*m+1], m < N.  Generic kernels, caller's stream.
template <typename T>
fc_status power_sequence(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, int b, double *spectrum, char *wsb) {
  const int start = kv->cu_seqlens[b];
  const int N = kv->cu_seqlens[b + 1] - start;
  if (N == 0) return FC_OK;
  const int d = kv->head_dim, H = kv->num_heads;
  const SeqPlan sp = plan_sequence(N, false);
  const ScoreLayout L = layout_for(h, sp, H, d);
  float2 *ws = reinterpret_cast<float2 *>(wsb + L.off_ws);
  float2 *spec = reinterpret_cast<float2 *>(wsb + L.off_spec);
  float2 *hhat = reinterpret_cast<float2 *>(wsb + L.off_hhat);
  float2 *hcol = reinterpret_cast<float2 *>(wsb + L.off_hcol);
  float2 *partial = reinterpret_cast<float2 *>(wsb + L.total);
  double *out = spectrum + 2 * (size_t)start;
  const T *kp = static_cast<const T *>(kv->k) + (long long)start * kv->stride_token;
  const T *vp = static_cast<const T *>(kv->v) + (long long)start * kv->stride_token;
  const FftPlan p1 = make_plan(sp.N1);
  fc_status s;
  if (sp.bluestein) {
    ChirpKernelLoader cl{N, sp.Nfft, -1};
    if ((s = launch_pass1(h, st, cl, sp, 8, 8, hcol, nullptr)) != FC_OK) return s;
    if ((s = launch_pass2<MID_SPEC>(h, st, sp, 8, 8, hcol, 0, hhat, 1.f)) != FC_OK) return s;
  }
  bool first = true;
  for (int h0 = 0; h0 < H; h0 += L.heads_per_group) {
    const int hg = (H - h0 < L.heads_per_group) ? H - h0 : L.heads_per_group;
    const int ncol_ws = hg * d;
    if (!sp.bluestein) {
      KvLoader<T, false> ld{kp, vp, kv->stride_token, kv->stride_head, h0, d, N, 0.f, 0.f};
      if ((s = launch_pass1(h, st, ld, sp, ncol_ws, sp.cs, ws, nullptr)) != FC_OK) return s;
      const FftPlan p2 = make_plan(sp.N2);
      const size_t sm = smem_pass2(sp, sp.cs2) + (size_t)sp.N2 * 2 * sizeof(float2);
      if ((s = set_smem(k_pass2_power, sm)) != FC_OK) return s;
      const int slices = ncol_ws / sp.cs2, ny = slices < kPowerNY ? slices : kPowerNY;
      k_pass2_power<<<dim3(sp.N1 / 2 + 1, ny), kThreads, sm, st>>>(p2, sp.N1, ncol_ws, ilog2(sp.cs2), ws, h->master,
                                                                   h->master_len, partial);
      if ((s = fc_after_launch(h)) != FC_OK) return s;
      k_power_accumulate<<<(N + 255) / 256, 256, 0, st>>>(partial, ny, N, out, first ? 1 : 0);
      if ((s = fc_after_launch(h)) != FC_OK) return s;
      first = false;
      continue;
    }
    const float invM = 1.f / (float)sp.Nfft;
    const int sub = L.sub_cols, cs = (sub % 64 == 0) ? sp.cs : 32;
    const int ngroups = (hg == 1) ? d / sub : 1;
    const int ncol = (hg == 1) ? sub : ncol_ws;
    int cs2 = 2 * sp.cs2 > 64 ? 64 : 2 * sp.cs2;
    while (ncol % cs2) cs2 >>= 1;
    const size_t sm3c = smem_pass13(sp, cs);
    for (int cg = 0; cg < ngroups; ++cg) {
      const int dd = (hg == 1) ? sub : d;
      KvLoader<T, true> ld{kp + cg * sub, vp + cg * sub, kv->stride_token, kv->stride_head, h0, dd, N, 0.f, 0.f};
      if ((s = launch_pass1(h, st, ld, sp, ncol, cs, ws, nullptr)) != FC_OK) return s;
      if ((s = launch_pass2<MID_MULH>(h, st, sp, ncol, cs2, ws, 0, hhat, invM)) != FC_OK) return s;
      if ((s = set_smem(k_pass3<EPI_SPEC, true>, sm3c)) != FC_OK) return s;
      k_pass3<EPI_SPEC, true><<<dim3(sp.N2, ncol / cs), kThreads, sm3c, st>>>(
          p1, sp.N2, N, ncol, ilog2(cs), ws, h->master, h->master_len, spec, nullptr, 0, dd, 0, 0.f, nullptr, 0.f, 0);
      if ((s = fc_after_launch(h)) != FC_OK) return s;
      k_spec_power<<<N / 2 + 1, kThreads, 0, st>>>(spec, ncol, N, partial);
      if ((s = fc_after_launch(h)) != FC_OK) return s;
      k_power_accumulate<<<(N + 255) / 256, 256, 0, st>>>(partial, 1, N, out, first ? 1 : 0);
      if ((s = fc_after_launch(h)) != FC_OK) return s;
      first = false;
    }
  }
  return FC_OK;
}

}  // namespace

extern "C" size_t fc_power_spectrum_workspace_bytes(const fc_handle *h, const fc_kv_view *kv) {
  if (validate_view(h, kv) != FC_OK) return 0;
  size_t need = 256;
  for (int b = 0; b < kv->batch; ++b) {
    const int N = kv->cu_seqlens[b + 1] - kv->cu_seqlens[b];
    if (N == 0) continue;
    const size_t t = layout_for(h, plan_sequence(N, false), kv->num_heads, kv->head_dim).total + power_partial_bytes(N);
    if (t > need) need = t;
  }
  return need;
}

extern "C" fc_status fc_power_spectrum(fc_handle *h, const fc_kv_view *kv, double *spectrum, void *workspace,
                                       size_t workspace_bytes, fc_stream stream) {
  fc_status s = validate_view(h, kv);
  if (s != FC_OK) return s;
  if (!spectrum) return FC_ERR_INVALID_ARG;
  const size_t need = fc_power_spectrum_workspace_bytes(h, kv);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return FC_ERR_WORKSPACE;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((s = fc_flush_pending(h, st)) != FC_OK) return s;     // the workspace may still be in use on the internal streams
  for (int b = 0; b < kv->batch && s == FC_OK; ++b) {
    switch (kv->dtype) {
      case FC_F32: s = power_sequence<float>(h, st, kv, b, spectrum, (char *)workspace); break;
      case FC_F16: s = power_sequence<__half>(h, st, kv, b, spectrum, (char *)workspace); break;
      default: s = power_sequence<__nv_bfloat16>(h, st, kv, b, spectrum, (char *)workspace); break;
    }
  }
  return s;
}

extern "C" fc_status fc_describe_plan(const fc_handle *h, int32_t seqlen, double gamma, int32_t out[4]) {
  if (!h || !out || seqlen < 1 || !(gamma >= 0.0 && gamma <= 1.0)) return FC_ERR_INVALID_ARG;
  if (seqlen > h->max_seqlen || (seqlen > 65536 && !is_pow2(seqlen))) return FC_ERR_UNSUPPORTED;
  const SeqPlan sp = plan_sequence(seqlen);
  out[0] = sp.bluestein ? 1 : 0;
  out[1] = sp.Nfft;
  out[2] = sp.N1;
  out[3] = sp.N2;
  if (sp.bluestein) {
    const ChirpChoice c = choose_chirp(h, sp, seqlen, cutoff_index(gamma, seqlen), true);
    out[0] = c.band >= 0 ? 2 : 1;
    out[1] = c.M;
    if (c.fast) {
      const ChirpShape cs = chirp_shape(c.M);
      out[2] = cs.n1();
      out[3] = cs.n2();
    }
  }
  return FC_OK;
}

extern "C" size_t fc_score_workspace_bytes(const fc_handle *h, const fc_kv_view *kv) {
  if (validate_view(h, kv) != FC_OK) return 0;
  size_t need = 256;
  for (int b = 0; b < kv->batch; ++b) {
    const int N = kv->cu_seqlens[b + 1] - kv->cu_seqlens[b];
    if (N == 0) continue;
    const ScoreLayout L = layout_for(h, plan_sequence(N, !h->generic_only), kv->num_heads, kv->head_dim);
    if (L.total > need) need = L.total;
  }
  return need;
}

extern "C" fc_status fc_score_layer(fc_handle *h, const fc_kv_view *kv, double gamma, float *scores,
                                    double *energy, void *workspace, size_t workspace_bytes,
                                    fc_stream stream) {
  fc_status s = validate_view(h, kv);
  if (s != FC_OK) return s;
  if (!scores || !energy) return FC_ERR_INVALID_ARG;
  if (!(gamma >= 0.0 && gamma <= 1.0)) return FC_ERR_INVALID_ARG;
  const size_t need = fc_score_workspace_bytes(h, kv);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return FC_ERR_WORKSPACE;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  claim_persisting_l2(h, kv, st);
  for (int b = 0; b < kv->batch && s == FC_OK; ++b) {
    switch (kv->dtype) {
      case FC_F32: s = score_sequence<float>(h, st, kv, b, gamma, scores, energy, (char *)workspace); break;
      case FC_F16: s = score_sequence<__half>(h, st, kv, b, gamma, scores, energy, (char *)workspace); break;
      default: s = score_sequence<__nv_bfloat16>(h, st, kv, b, gamma, scores, energy, (char *)workspace); break;
    }
  }
  return s;
}

// ---------------------------------------------------------------------------
// fc_cutoff_from_spectrum: the smallest omega whose kept band holds a given share of the energy.
// One block per sequence; thread t adds up a contiguous run of bins, a block scan of the run totals in
// fp64 finds the run in which the running sum first reaches share * total, and the thread that owns the
// run walks it.  Sums are taken in a fixed order (deterministic).
// ---------------------------------------------------------------------------
namespace {

constexpr int kCutThreads = 1024;
struct CutTable { int start[65]; };

__global__ void __launch_bounds__(kCutThreads)
k_cutoff_from_spectrum(const double *__restrict__ spectrum, const __grid_constant__ CutTable st, int b0, double share,
                       int *__restrict__ omega, double *__restrict__ gamma) {
  __shared__ double run[kCutThreads];
  __shared__ double s_total;
  const int tid = threadIdx.x;
  const int s0 = st.start[blockIdx.x], N = st.start[blockIdx.x + 1] - s0;
  const int b = b0 + blockIdx.x;
  if (N == 0) {
    if (tid == 0) { omega[b] = 0; gamma[b] = 0.0; }
    return;
  }
  const int per = (N + kCutThreads - 1) / kCutThreads;
  const int lo = tid * per, hi = lo + per < N ? lo + per : N;
  const double *P = spectrum + 2 * (size_t)s0;
  double mine = 0.0;
  for (int m = lo; m < hi; ++m) mine += P[2 * m] + P[2 * m + 1];
  run[tid] = mine;
  __syncthreads();
  // inclusive scan of the run totals (Hillis-Steele, fp64)
  for (int o = 1; o < kCutThreads; o <<= 1) {
    const double add = tid >= o ? run[tid - o] : 0.0;
    __syncthreads();
    run[tid] += add;
    __syncthreads();
  }
  if (tid == kCutThreads - 1) s_total = run[tid];
  __syncthreads();
  const double total = s_total, want = share * total;
  if (!(total > 0.0)) {
    if (tid == 0) { omega[b] = 0; gamma[b] = 0.5 / (double)N; }
    return;
  }
  // the run that holds the crossing: the first non-empty one whose running sum has reached `want` (the
  // scan's sums of one and the same set can differ in the last bit, so "the last run reaches the total"
  // is not relied on: without a qualifying run the last non-empty one is taken)
  __shared__ int s_owner;
  if (tid == 0) s_owner = kCutThreads;
  __syncthreads();
  if (lo < hi && run[tid] >= want) atomicMin(&s_owner, tid);
  __syncthreads();
  const int owner = s_owner < kCutThreads ? s_owner : (N - 1) / per;
  if (tid == owner) {
    double acc = run[tid] - mine;
    int m = lo;
    for (; m < hi; ++m) {
      acc += P[2 * m] + P[2 * m + 1];
      if (acc >= want) break;
    }
    if (m >= hi) m = hi - 1;
    omega[b] = m;
    gamma[b] = ((double)m + 0.5) / (double)N;
  }
}

}  // namespace

extern "C" fc_status fc_cutoff_from_spectrum(fc_handle *h, const double *spectrum, int32_t batch,
                                             const int32_t *cu_seqlens, double share, int32_t *omega,
                                             double *gamma, fc_stream stream) {
  if (!h || !spectrum || !cu_seqlens || !omega || !gamma || batch < 0) return FC_ERR_INVALID_ARG;
  if (!(share >= 0.0 && share <= 1.0) || cu_seqlens[0] != 0) return FC_ERR_INVALID_ARG;
  for (int b = 0; b < batch; ++b)
    if (cu_seqlens[b + 1] < cu_seqlens[b]) return FC_ERR_INVALID_ARG;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  fc_status s;
  for (int b0 = 0; b0 < batch; b0 += 64) {
    const int nseq = batch - b0 < 64 ? batch - b0 : 64;
    CutTable tab;
    for (int i = 0; i <= nseq; ++i) tab.start[i] = cu_seqlens[b0 + i];
    k_cutoff_from_spectrum<<<nseq, kCutThreads, 0, st>>>(spectrum, tab, b0, share, omega, gamma);
    if ((s = fc_after_launch(h)) != FC_OK) return s;
  }
  return FC_OK;
}

// ---------------------------------------------------------------------------
// fc_score_layer_static: the same scoring with every byte of scratch in arrays that are
// part of the loaded library image, for callers that must not allocate device memory.
// ---------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxSeqlen = 4096;                       // longest sequence accepted
constexpr int kStaticMasterLen = 4 * kStaticMaxSeqlen;       // same sizing rule as fc_create's table
constexpr size_t kStaticScratchBytes = FC_STATIC_SCRATCH_BYTES;

// Scratch shared by every call of fc_score_layer_static on a device; it keeps whatever the
// last call left there.  The kernels below write each region before they read it, so
// nothing has to be cleared between calls.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static __device__ __align__(256) float2 g_static_master[kStaticMasterLen];
static __device__ int g_static_status;
static __device__ unsigned g_static_counter;

// exp(-2*pi*j*i/len) in fp64, rounded once to fp32 (same definition as the handle's table).
__global__ void k_fill_static_master(float2 *master, int len) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= len) return;
  double s, c;
  sincospi(-2.0 * (double)i / (double)len, &s, &c);
  master[i] = make_float2((float)c, (float)s);
}

// Device addresses of the arrays above, looked up once per device.  In host code the
// array names stand for the symbols, not for device memory: they must never be passed
// to a kernel; cudaGetSymbolAddress gives the pointer a kernel can use.
struct StaticSetup {
  bool ready;
  unsigned char *scratch;
  float2 *master;
  int *status;
  unsigned *counter;
  int num_sms;
};
constexpr int kMaxDevices = 64;
StaticSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

fc_status static_setup(int dev, StaticSetup *out) {
  if (dev < 0 || dev >= kMaxDevices) return FC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  StaticSetup &s = g_setup[dev];
  if (!s.ready) {
    void *p_scratch = nullptr, *p_master = nullptr, *p_status = nullptr, *p_counter = nullptr;
    FC_CUDA_TRY(cudaGetSymbolAddress(&p_scratch, g_static_scratch));
    FC_CUDA_TRY(cudaGetSymbolAddress(&p_master, g_static_master));
    FC_CUDA_TRY(cudaGetSymbolAddress(&p_status, g_static_status));
    FC_CUDA_TRY(cudaGetSymbolAddress(&p_counter, g_static_counter));
    k_fill_static_master<<<(kStaticMasterLen + 255) / 256, 256>>>(static_cast<float2 *>(p_master), kStaticMasterLen);
    FC_CUDA_TRY(cudaGetLastError());
    FC_CUDA_TRY(cudaDeviceSynchronize());
    s.scratch = static_cast<unsigned char *>(p_scratch);
    s.master = static_cast<float2 *>(p_master);
    s.status = static_cast<int *>(p_status);
    s.counter = static_cast<unsigned *>(p_counter);
    FC_CUDA_TRY(cudaDeviceGetAttribute(&s.num_sms, cudaDevAttrMultiProcessorCount, dev));
    s.ready = true;
  }
  *out = s;
  return FC_OK;
}

}  // namespace

extern "C" size_t fc_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" fc_status fc_score_layer_static(const fc_kv_view *kv, double gamma, float *scores,
                                           double *energy, fc_stream stream) {
  if (!kv || !scores || !energy) return FC_ERR_INVALID_ARG;
  if (!(gamma >= 0.0 && gamma <= 1.0)) return FC_ERR_INVALID_ARG;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  StaticSetup su;
  fc_status s = static_setup(dev, &su);
  if (s != FC_OK) return s;
  // A handle that lives on this stack frame and owns nothing: its table, status word and
  // counter are the static arrays, and it is restricted to the single-stream kernels.
  fc_handle hs = {};
  hs.device = dev;
  hs.max_seqlen = kStaticMaxSeqlen;
  hs.master_len = kStaticMasterLen;
  hs.master = su.master;
  hs.status_word = su.status;
  hs.done_counter = su.counter;
  hs.group_bytes = 1;                 // one head per transform group: the smallest workspace
  hs.tune_cpw = 32;
  hs.tune_cp = 8;
  hs.prof_class = FC_K_NONE;
  hs.generic_only = true;
  hs.num_sms = su.num_sms;
  s = validate_view(&hs, kv);         // lengths above kStaticMaxSeqlen come back as FC_ERR_UNSUPPORTED
  if (s != FC_OK) return s;
  const size_t need = fc_score_workspace_bytes(&hs, kv);
  if (need == 0) return FC_ERR_INVALID_ARG;
  if (need > kStaticScratchBytes) return FC_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  for (int b = 0; b < kv->batch && s == FC_OK; ++b) {
    switch (kv->dtype) {
      case FC_F32: s = score_sequence<float>(&hs, st, kv, b, gamma, scores, energy, (char *)su.scratch); break;
      case FC_F16: s = score_sequence<__half>(&hs, st, kv, b, gamma, scores, energy, (char *)su.scratch); break;
      default: s = score_sequence<__nv_bfloat16>(&hs, st, kv, b, gamma, scores, energy, (char *)su.scratch); break;
    }
  }
  return s;
}

extern "C" fc_status fc_static_last_device_status(fc_stream stream) {
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  StaticSetup su;
  fc_status s = static_setup(dev, &su);
  if (s != FC_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FC_CUDA_TRY(cudaStreamSynchronize(st));
  int word = 0;
  FC_CUDA_TRY(cudaMemcpy(&word, su.status, sizeof(int), cudaMemcpyDeviceToHost));
  if (word != 0) FC_CUDA_TRY(cudaMemset(su.status, 0, sizeof(int)));
  if (word == 0) return FC_OK;
  return (word & FC_DEV_FLAG_INTERNAL) ? FC_ERR_INTERNAL : FC_ERR_TIMEOUT;
}
