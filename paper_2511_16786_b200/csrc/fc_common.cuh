// Shared device helpers of the FlashCache kernels: complex arithmetic on float2,
// register-resident radix-2/4/8/16 DFTs, and the batched in-shared-memory FFT
// stages.  The transforms here run along the token axis with the channels of a
// tile spread across the lanes of a warp, so every lane of a warp executes the
// same butterfly with the same twiddle and shared-memory rows are read with
// unit stride.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "../../include/flashcache.h"

#define FC_MAX_STAGES 4
#define FC_MAX_AUX 4     // internal streams a handle may use
#define FC_HHAT_SLOTS 8  // chirp-kernel spectra a handle keeps (one per sequence length)

// Bits of the device status word.
#define FC_DEV_FLAG_INTERNAL 1
#define FC_DEV_FLAG_TIMEOUT 2

struct fc_handle {
  int device;
  int max_seqlen;
  int master_len;          // power of two; master[i] = exp(-2*pi*i*j/master_len)
  float2 *master;          // DEVICE
  int *status_word;        // DEVICE
  unsigned *done_counter;  // DEVICE, zero between calls (the last block of a sequence resets it)
  size_t group_bytes;
  int tune_cpw, tune_cp;   // tile widths of the specialised kernels (channel pairs), see fc_create
  int num_sms;
  // L2 residency of the transform intermediates: the per-stream workspace buffers are declared a
  // persisting access window on the internal streams (0 switches it off, fc_set_l2_persist)
  int l2_persist;
  int persist_on;                      // the context's persisting-L2 set-aside is currently claimed by this handle
  size_t persist_max, window_max;      // device limits (bytes)
  const void *window_base[FC_MAX_AUX]; // what each internal stream's window was last set to
  size_t window_bytes[FC_MAX_AUX];
  unsigned long long launches;
  // internal streams: consecutive head groups of one fc_score_layer call are transformed
  // concurrently, round robin over the streams, each with its own workspace buffer
  cudaStream_t aux[FC_MAX_AUX];
  int num_aux;             // how many of them are used (2 by default, fc_set_internal_streams)
  cudaEvent_t ev_fork, ev_join[FC_MAX_AUX];
  // optional per-kernel-class timing (fc_profile_begin / fc_profile_end)
  int prof_class;
  cudaEvent_t *prof_events;   // pairs
  int prof_cap, prof_used;
  int prof_stride, prof_seen;  // every prof_stride-th launch of the class is timed
  // true only for the stack handle of fc_score_layer_static: every length takes the generic
  // single-stream kernels (no internal streams or events exist there)
  bool generic_only;
  int select_overlap;      // 1: consecutive fc_select_compact launches may overlap (fc_set_select_overlap)
  // fc_set_score_overlap: consecutive fc_score_layer calls keep running on the two internal streams
  // without rejoining the caller's stream; the join is made by the next call that consumes their results
  int score_overlap;
  int band_form;           // 1: the chirp path may use its band form (fc_set_chirp_band)
  unsigned step;                 // specialised-path sequences scored so far (parity picks partial-sum buffers)
  long long last_sig;            // (N, heads, head_dim) of the previous specialised-path step
  bool pending_join;             // internal streams hold work the caller's stream has not waited for
  cudaEvent_t ev_done[2][FC_MAX_AUX];   // [step parity][internal stream]: that stream finished that step
  // fc_compress_host (created on its first call): the stream the host-to-device copies run on, one
  // event per layer (that layer's copies have landed), and the point of the previous job after
  // which the staged inputs of its arena may be overwritten
  // spectra of the chirp kernel of the last FC_HHAT_SLOTS sequence lengths that took the chirp path (DEVICE,
  // allocated by fc_create: FC_HHAT_SLOTS x hhat_cache_len points; hhat_cache_n[i] = length in slot i, 0 = none;
  // slots are reused round robin)
  float2 *hhat_cache;
  int hhat_cache_len, hhat_cache_next;
  int hhat_slot_len;       // points per slot: the spectrum (hhat_cache_len) and 2N per-row chirp factors behind it
  long long hhat_cache_n[FC_HHAT_SLOTS];   // key of slot i: length + ((band + 1) << 32), 0 = none
  cudaStream_t host_copy;
  cudaEvent_t *host_ev;
  int host_ev_cap;
  cudaEvent_t ev_inputs_free;
  cudaEvent_t ev_outputs_done;      // the previous fc_compress_host job has copied its rows back to the host
  const void *host_last_arena;
};

// Kernel classes for fc_profile_begin.
enum { FC_K_NONE = 0, FC_K_PASS1 = 1, FC_K_PASS2 = 2, FC_K_PASS3 = 3, FC_K_SELECT = 4, FC_K_GATHER = 5, FC_K_OTHER = 6 };

// Brackets one launch with an event pair when its class is being profiled.
struct ProfScope {
  fc_handle *h;
  cudaStream_t st;
  bool on;
  ProfScope(fc_handle *h_, int cls, cudaStream_t st_) : h(h_), st(st_) {
    on = h->prof_class == cls && h->prof_used < h->prof_cap && (h->prof_seen++ % h->prof_stride) == 0;
    if (on) cudaEventRecord(h->prof_events[2 * h->prof_used], st);
  }
  ~ProfScope() {
    if (on) {
      cudaEventRecord(h->prof_events[2 * h->prof_used + 1], st);
      h->prof_used++;
    }
  }
};

// Radix plan of one power-of-two FFT length: len = prod radix[s].
struct FftPlan {
  int len;
  int nstages;
  int radix[FC_MAX_STAGES];
};

__host__ inline FftPlan make_plan(int len) {
  FftPlan p;
  p.len = len;
  int bits = 0;
  while ((1 << bits) < len) ++bits;
  p.nstages = (bits + 3) / 4;
  for (int s = 0; s < FC_MAX_STAGES; ++s) p.radix[s] = 1;
  int left = bits;
  for (int s = 0; s < p.nstages; ++s) {
    int take = (left + (p.nstages - s) - 1) / (p.nstages - s);   // spread the bits evenly, larger first
    p.radix[s] = 1 << take;
    left -= take;
  }
  return p;
}

// ------------------------------------------------------------------ complex
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 w) {
  return make_float2(a.x * w.x - a.y * w.y, a.x * w.y + a.y * w.x);
}
__device__ __forceinline__ float2 cmul_conj(float2 a, float2 w) {   // a * conj(w)
  return make_float2(a.x * w.x + a.y * w.y, a.y * w.x - a.x * w.y);
}
__device__ __forceinline__ float2 cconj(float2 a) { return make_float2(a.x, -a.y); }
__device__ __forceinline__ float2 cscale(float2 a, float s) { return make_float2(a.x * s, a.y * s); }

// multiply by exp(DIR * j*pi/2): DIR=-1 -> -j, DIR=+1 -> +j
template <int DIR>
__device__ __forceinline__ float2 mul_j(float2 a) {
  return DIR < 0 ? make_float2(a.y, -a.x) : make_float2(-a.y, a.x);
}

// ------------------------------------------------------------------ small DFTs
// y[k] = sum_n x[n] exp(DIR*2*pi*j*n*k/R), natural order in and out.
template <int DIR>
__device__ __forceinline__ void dft2(float2 &a, float2 &b) {
  float2 t = a;
  a = cadd(t, b);
  b = csub(t, b);
}

template <int DIR>
__device__ __forceinline__ void dft4(float2 &a0, float2 &a1, float2 &a2, float2 &a3) {
  float2 s0 = cadd(a0, a2), d0 = csub(a0, a2);
  float2 s1 = cadd(a1, a3), d1 = mul_j<DIR>(csub(a1, a3));
  a0 = cadd(s0, s1);
  a2 = csub(s0, s1);
  a1 = cadd(d0, d1);
  a3 = csub(d0, d1);
}

template <int DIR>
__device__ __forceinline__ void dft8(float2 (&x)[8]) {
  const float h = 0.70710678118654752440f;
  dft4<DIR>(x[0], x[2], x[4], x[6]);   // even samples -> x[0],x[2],x[4],x[6] = E0..E3
  dft4<DIR>(x[1], x[3], x[5], x[7]);   // odd samples  -> x[1],x[3],x[5],x[7] = O0..O3
  float2 e0 = x[0], e1 = x[2], e2 = x[4], e3 = x[6];
  float2 o0 = x[1], o1 = x[3], o2 = x[5], o3 = x[7];
  // w8^1 = (1 + DIR*j)/sqrt2, w8^2 = DIR*j, w8^3 = (-1 + DIR*j)/sqrt2
  float2 t1 = DIR < 0 ? make_float2((o1.x + o1.y) * h, (o1.y - o1.x) * h)
                      : make_float2((o1.x - o1.y) * h, (o1.x + o1.y) * h);
  float2 t2 = mul_j<DIR>(o2);
  float2 t3 = DIR < 0 ? make_float2((o3.y - o3.x) * h, -(o3.x + o3.y) * h)
                      : make_float2(-(o3.x + o3.y) * h, (o3.x - o3.y) * h);
  x[0] = cadd(e0, o0); x[4] = csub(e0, o0);
  x[1] = cadd(e1, t1); x[5] = csub(e1, t1);
  x[2] = cadd(e2, t2); x[6] = csub(e2, t2);
  x[3] = cadd(e3, t3); x[7] = csub(e3, t3);
}

template <int DIR>
__device__ __forceinline__ void dft16(float2 (&x)[16]) {
  const float c1 = 0.92387953251128675613f, s1 = 0.38268343236508977173f;
  const float h = 0.70710678118654752440f;
  float2 e[8], o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { e[i] = x[2 * i]; o[i] = x[2 * i + 1]; }
  dft8<DIR>(e);
  dft8<DIR>(o);
  const float sg = DIR < 0 ? -1.f : 1.f;
  // w16^k = (cos(k*pi/8), DIR*sin(k*pi/8))
  float2 t[8];
  t[0] = o[0];
  t[1] = cmul(o[1], make_float2(c1, sg * s1));
  t[2] = cmul(o[2], make_float2(h, sg * h));
  t[3] = cmul(o[3], make_float2(s1, sg * c1));
  t[4] = mul_j<DIR>(o[4]);
  t[5] = cmul(o[5], make_float2(-s1, sg * c1));
  t[6] = cmul(o[6], make_float2(-h, sg * h));
  t[7] = cmul(o[7], make_float2(-c1, sg * s1));
#pragma unroll
  for (int k = 0; k < 8; ++k) { x[k] = cadd(e[k], t[k]); x[k + 8] = csub(e[k], t[k]); }
}

// Odd lengths by the symmetric form: with a_m = x[m] + x[P-m], b_m = x[m] - x[P-m],
//   y[k], y[P-k] = x[0] + sum_m cos(2*pi*k*m/P) a_m  +/-  DIR*j * sum_m sin(2*pi*k*m/P) b_m.
template <int DIR>
__device__ __forceinline__ void dft3(float2 &x0, float2 &x1, float2 &x2) {
  const float s = 0.86602540378443864676f;
  const float2 a = cadd(x1, x2), b = csub(x1, x2);
  const float2 r = make_float2(fmaf(-0.5f, a.x, x0.x), fmaf(-0.5f, a.y, x0.y));
  const float2 i = mul_j<DIR>(cscale(b, s));
  x0 = cadd(x0, a);
  x1 = cadd(r, i);
  x2 = csub(r, i);
}

template <int DIR>
__device__ __forceinline__ void dft5(float2 (&x)[5]) {
  const float c1 = 0.30901699437494742410f, c2 = -0.80901699437494742410f;
  const float s1 = 0.95105651629515357212f, s2 = 0.58778525229247312917f;
  const float2 a1 = cadd(x[1], x[4]), a2 = cadd(x[2], x[3]), b1 = csub(x[1], x[4]), b2 = csub(x[2], x[3]);
  const float2 r1 = make_float2(fmaf(c1, a1.x, fmaf(c2, a2.x, x[0].x)), fmaf(c1, a1.y, fmaf(c2, a2.y, x[0].y)));
  const float2 r2 = make_float2(fmaf(c2, a1.x, fmaf(c1, a2.x, x[0].x)), fmaf(c2, a1.y, fmaf(c1, a2.y, x[0].y)));
  const float2 i1 = mul_j<DIR>(make_float2(fmaf(s1, b1.x, s2 * b2.x), fmaf(s1, b1.y, s2 * b2.y)));
  const float2 i2 = mul_j<DIR>(make_float2(fmaf(s2, b1.x, -s1 * b2.x), fmaf(s2, b1.y, -s1 * b2.y)));
  x[0] = cadd(x[0], cadd(a1, a2));
  x[1] = cadd(r1, i1); x[4] = csub(r1, i1);
  x[2] = cadd(r2, i2); x[3] = csub(r2, i2);
}

template <int DIR>
__device__ __forceinline__ void dft7(float2 (&x)[7]) {
  // cos and sin of 2*pi*i/7, i = 1..3
  const float c[3] = {0.62348980185873353053f, -0.22252093395631440429f, -0.90096886790241912624f};
  const float s[3] = {0.78183148246802980871f, 0.97492791218182360702f, 0.43388373911755812048f};
  float2 a[3], b[3];
#pragma unroll
  for (int m = 0; m < 3; ++m) { a[m] = cadd(x[m + 1], x[6 - m]); b[m] = csub(x[m + 1], x[6 - m]); }
  const float2 x0 = x[0];
  x[0] = cadd(x0, cadd(a[0], cadd(a[1], a[2])));
#pragma unroll
  for (int k = 1; k <= 3; ++k) {
    float2 r = x0, im = make_float2(0.f, 0.f);
#pragma unroll
    for (int m = 1; m <= 3; ++m) {
      const int idx = (k * m) % 7;                       // 1..6; cos is even, sin odd about 7/2
      const float cc = idx <= 3 ? c[idx - 1] : c[6 - idx];
      const float ss = idx <= 3 ? s[idx - 1] : -s[6 - idx];
      r = make_float2(fmaf(cc, a[m - 1].x, r.x), fmaf(cc, a[m - 1].y, r.y));
      im = make_float2(fmaf(ss, b[m - 1].x, im.x), fmaf(ss, b[m - 1].y, im.y));
    }
    const float2 i = mul_j<DIR>(im);
    x[k] = cadd(r, i);
    x[7 - k] = csub(r, i);
  }
}

template <int R, int DIR>
__device__ __forceinline__ void dft_small(float2 (&x)[R]);

// R = R1*R2 with coprime factors (prime-factor mapping, no twiddles between the two stages):
// input n = (n1*R2 + n2*R1) mod R, output k with k = k1 (mod R1) and k = k2 (mod R2).
template <int R1, int R2, int DIR>
__device__ __forceinline__ void dft_coprime(float2 (&x)[R1 * R2]) {
  constexpr int R = R1 * R2;
  float2 t[R1][R2];
#pragma unroll
  for (int n1 = 0; n1 < R1; ++n1) {
#pragma unroll
    for (int n2 = 0; n2 < R2; ++n2) t[n1][n2] = x[(n1 * R2 + n2 * R1) % R];
    dft_small<R2, DIR>(t[n1]);
  }
#pragma unroll
  for (int k2 = 0; k2 < R2; ++k2) {
    float2 col[R1];
#pragma unroll
    for (int n1 = 0; n1 < R1; ++n1) col[n1] = t[n1][k2];
    dft_small<R1, DIR>(col);
#pragma unroll
    for (int k1 = 0; k1 < R1; ++k1) {
      int k = k1;                                        // smallest k = k1 (mod R1) with k = k2 (mod R2)
#pragma unroll
      for (int i = 0; i < R2; ++i) if (k % R2 != k2) k += R1;
      x[k] = col[k1];
    }
  }
}

template <int R, int DIR>
__device__ __forceinline__ void dft_small(float2 (&x)[R]) {
  if constexpr (R == 2) dft2<DIR>(x[0], x[1]);
  else if constexpr (R == 3) dft3<DIR>(x[0], x[1], x[2]);
  else if constexpr (R == 4) dft4<DIR>(x[0], x[1], x[2], x[3]);
  else if constexpr (R == 5) dft5<DIR>(x);
  else if constexpr (R == 7) dft7<DIR>(x);
  else if constexpr (R == 8) dft8<DIR>(x);
  else if constexpr (R == 10) dft_coprime<2, 5, DIR>(x);
  else if constexpr (R == 12) dft_coprime<4, 3, DIR>(x);
  else if constexpr (R == 14) dft_coprime<2, 7, DIR>(x);
  else {
    static_assert(R == 16, "unsupported small DFT length");
    dft16<DIR>(x);
  }
}

// ------------------------------------------------------------------ batched stages in shared memory
// Tile S[len][ncol] (ncol a power of two, column index fastest).  tw[i] =
// exp(-2*pi*j*i/len).  One radix-R stage over blocks of length Ls:
//   forward (decimation in frequency): butterfly, then multiply output p by w_Ls^(j*p);
//   inverse (decimation in time, the exact mirror): multiply input p by conj(w_Ls^(j*p)), butterfly.
// A forward pass over all stages leaves bin rev(pos) at row pos; the inverse pass
// takes that order back to natural order.  No 1/len factor is applied.
template <int R, bool INVERSE>
__device__ __forceinline__ void fft_stage(float2 *S, int ncol_log2, int len, int Ls,
                                          const float2 *tw, int tid, int nthreads) {
  const int sub = Ls / R;
  const int ncol = 1 << ncol_log2;
  const int total = (len / R) << ncol_log2;
  const int twstep = len / Ls;
  for (int w = tid; w < total; w += nthreads) {
    const int c = w & (ncol - 1);
    const int b = w >> ncol_log2;
    const int block = b / sub;
    const int j = b - block * sub;
    float2 *base = S + ((size_t)(block * Ls + j) << ncol_log2) + c;
    const int stride = sub << ncol_log2;
    float2 x[R];
#pragma unroll
    for (int p = 0; p < R; ++p) x[p] = base[p * stride];
    if (INVERSE) {
      if (sub > 1) {
#pragma unroll
        for (int p = 1; p < R; ++p) x[p] = cmul_conj(x[p], tw[j * p * twstep]);
      }
      dft_small<R, +1>(x);
    } else {
      dft_small<R, -1>(x);
      if (sub > 1) {
#pragma unroll
        for (int p = 1; p < R; ++p) x[p] = cmul(x[p], tw[j * p * twstep]);
      }
    }
#pragma unroll
    for (int p = 0; p < R; ++p) base[p * stride] = x[p];
  }
}

template <bool INVERSE>
__device__ __forceinline__ void fft_stage_dyn(int R, float2 *S, int ncol_log2, int len, int Ls,
                                              const float2 *tw, int tid, int nthreads) {
  switch (R) {
    case 16: fft_stage<16, INVERSE>(S, ncol_log2, len, Ls, tw, tid, nthreads); break;
    case 8: fft_stage<8, INVERSE>(S, ncol_log2, len, Ls, tw, tid, nthreads); break;
    case 4: fft_stage<4, INVERSE>(S, ncol_log2, len, Ls, tw, tid, nthreads); break;
    case 2: fft_stage<2, INVERSE>(S, ncol_log2, len, Ls, tw, tid, nthreads); break;
    default: break;
  }
}

// All forward stages, natural order -> digit-reversed order.  Ends with __syncthreads().
__device__ __forceinline__ void fft_forward_tile(const FftPlan &plan, float2 *S, int ncol_log2,
                                                 const float2 *tw, int tid, int nthreads) {
  int Ls = plan.len;
  for (int s = 0; s < plan.nstages; ++s) {
    fft_stage_dyn<false>(plan.radix[s], S, ncol_log2, plan.len, Ls, tw, tid, nthreads);
    Ls /= plan.radix[s];
    __syncthreads();
  }
}

// All inverse stages, digit-reversed order -> natural order.  Ends with __syncthreads().
__device__ __forceinline__ void fft_inverse_tile(const FftPlan &plan, float2 *S, int ncol_log2,
                                                 const float2 *tw, int tid, int nthreads) {
  int Ls = 1;
  for (int s = plan.nstages - 1; s >= 0; --s) {
    Ls *= plan.radix[s];
    fft_stage_dyn<true>(plan.radix[s], S, ncol_log2, plan.len, Ls, tw, tid, nthreads);
    __syncthreads();
  }
}

// Bin held at row pos after the forward stages.
__device__ __forceinline__ int digit_rev(const FftPlan &plan, int pos) {
  int k = 0, mult = 1, rem = plan.len;
  for (int s = 0; s < plan.nstages; ++s) {
    const int R = plan.radix[s];
    const int sub = rem / R;
    const int p = pos / sub;
    pos -= p * sub;
    k += p * mult;
    mult *= R;
    rem = sub;
  }
  return k;
}

// Row that holds bin k after the forward stages.
__device__ __forceinline__ int digit_pos(const FftPlan &plan, int k) {
  int pos = 0, rem = plan.len;
  for (int s = 0; s < plan.nstages; ++s) {
    const int R = plan.radix[s];
    const int sub = rem / R;
    const int p = k % R;
    k /= R;
    pos += p * sub;
    rem = sub;
  }
  return pos;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Host-side launch bookkeeping shared by the translation units.
#define FC_CUDA_TRY(expr)                          \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return FC_ERR_CUDA;    \
  } while (0)

// Makes `st` wait for everything the internal streams were given (no-op when nothing is pending).
inline fc_status fc_flush_pending(fc_handle *h, cudaStream_t st) {
  if (!h->pending_join) return FC_OK;
  for (int i = 0; i < h->num_aux; ++i) {
    FC_CUDA_TRY(cudaEventRecord(h->ev_join[i], h->aux[i]));
    FC_CUDA_TRY(cudaStreamWaitEvent(st, h->ev_join[i], 0));
  }
  h->pending_join = false;
  return FC_OK;
}

// After every launch: takes (and so clears) the runtime's pending error, so a failed launch is reported by
// the call that made it and does not linger for the caller's next CUDA call.
inline fc_status fc_after_launch(fc_handle *h) {
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? FC_OK : FC_ERR_CUDA;
}

// Shared claim on the context's persisting-L2 limit (fc_api.cu).
bool fc_persist_acquire(fc_handle *h);
void fc_persist_release(fc_handle *h);
