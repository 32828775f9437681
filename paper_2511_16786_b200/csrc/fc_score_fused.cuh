// Fused, persistent form of the three transform passes for power-of-two sequence
// lengths N = N1*N2 from 4096 to 65536 (N1 = 16*R1B, N2 = 16*R2B).  Same mathematics
// as fc_score.cu (see the header comment there); what differs:
//
//  * ONE launch scores a whole (layer, sequence).  The columns of the layer are cut into
//    units of UC complex columns (about 8 MB of intermediate each); stage s consists of
//    the pass-1 tiles of unit s, then the pass-2 tiles of unit s-1, then the pass-3 tiles
//    of unit s-2.  Persistent blocks take tiles in that order from an atomic counter and
//    wait (bounded) on per-unit completion counters, so a tile only ever waits for
//    tiles that were handed out before it; a producer and its first consumer are three
//    tile blocks apart, more than the blocks in flight, so the wait is normally over
//    before it starts.  The intermediates live in a ring of unit slots that stays in L2.
//  * every tile is 4096 complex points = 2048 float4 (32 KB), processed by the 128 threads of
//    four compute warps; a fifth (scheduler) warp asks for tile numbers, waits for the tiles
//    they depend on, fills the second shared-memory buffer through the TMA unit while the current
//    one is transformed in place, and reports finished tiles, so the compute warps only ever
//    wait for a full buffer (mbarrier).
//  * pass 3 writes one partial score per 2*CPW channels; the block that delivers the last
//    partial of a (head, row set) adds them in a fixed order (deterministic).
//  * a thread owns two adjacent channels as ONE packed value per component:
//    float4 = (re_a, re_b, im_a, im_b), and all butterflies run on the packed
//    fp32x2 add/mul/fma instructions of sm_100, halving the issue slots of the
//    arithmetic.
//
// The transform is unnormalised (factor N); pass 3 folds 1/N^2 into the score.
#pragma once
#include <cuda.h>   // CUtensorMap (type only; the encoder is looked up at run time)

#include "fc_common.cuh"

namespace fused {

constexpr int NT = 128;        // threads per block
constexpr int TILE4 = 2048;    // float4 per tile
constexpr int BUF4 = TILE4;     // float4 per shared-memory buffer

// Scheduler state in global memory (owned by the handle, all zero between launches).
struct Sched {
  unsigned tile_counter;
  unsigned exit_counter;
  unsigned abort_flag;
  unsigned pad;
  unsigned done1[1024];   // pass-1 tiles finished per unit
  unsigned done2[1024];   // pass-2 tiles finished per unit
  unsigned done3[1024];   // pass-3 tiles finished per unit
  unsigned cnt3[65536];   // partial scores delivered per (head, n2); the last deliverer resets its entry
  // running totals since the handle was created (diagnostic, see fc_fused_stats): tiles, tiles whose
  // dependencies were not finished when the scheduler warp first looked, unused, clock cycles of thread 0
  // inside pass-1 / pass-2 / pass-3 tiles, cycles waiting for a full buffer, cycles in the tile loop
  unsigned long long stats[8];
  // scheduler warp (lane 0, summed): cycles waiting for a buffer to come back, waiting for dependencies,
  // issuing the loads; compute warps: cycles from the end of the issue to the buffer being full
  unsigned long long stats2[4];
};
constexpr int kMaxCnt3 = 65536;

struct Params {
  const void *k, *v;               // first token of the sequence
  long long stride_token_b, stride_head_b;   // bytes
  int N, omega, head_dim, num_heads;
  int UC, U, R, lag;               // unit columns, units, ring slots, stages between the passes of a unit
  int TPU, ncb1, ncb2;             // tiles per unit and pass; column blocks per unit in pass 1/3 and in pass 2
  int nparts;                      // partial scores per (head, token) = head_dim / (2*CPW)
  unsigned total_tiles;
  float2 *ws;                      // ring of R unit slots, each [N1*N2][UC] float2 (stored as planar pairs)
  const float2 *master;
  int master_len;
  float *partial;                  // [nparts][num_heads][N] partial scores (used when nparts > 1)
  float *scores;                   // already offset to the sequence's first token
  long long score_stride;          // tokens in the packed batch
  float inv_scale;                 // 1 / (N^2 d)
  double *part_tot, *part_hi;      // per-tile energy partial sums
  double *energy;                  // [4]
  Sched *sched;
  int *status;
  unsigned spin_limit;
};

// Tensor maps of one launch (encoded on the host, read by the TMA unit):
//   k, v   K / V of the sequence as [N1/2 groups][2*N2 tokens][heads][channels]; a box is one channel
//          slice of the N1/2 tokens that share a position inside their group (one half of a pass-1 tile)
//   ws2    the ring as [R*N1 rows k1][N2][2*UC floats], box = N2 x (4*CP floats): one half of a pass-2 tile
//   ws3    the same tensor, box = N1 x 1 x (4*CPW floats): a pass-3 tile
struct TmaMaps { CUtensorMap k, v, ws2, ws3; };

// ------------------------------------------------------------------ packed arithmetic
// Two complex numbers a and b (adjacent channels): r = (re_a, re_b), i = (im_a, im_b).
struct c2 { float2 r, i; };

__device__ __forceinline__ float2 padd(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 psub(float2 a, float2 b) { return __ffma2_rn(b, make_float2(-1.f, -1.f), a); }
__device__ __forceinline__ float2 pmul(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 pfma(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 bc(float s) { return make_float2(s, s); }

__device__ __forceinline__ c2 cadd2(const c2 &a, const c2 &b) { return {padd(a.r, b.r), padd(a.i, b.i)}; }
__device__ __forceinline__ c2 csub2(const c2 &a, const c2 &b) { return {psub(a.r, b.r), psub(a.i, b.i)}; }
__device__ __forceinline__ c2 from4(float4 t) { return {make_float2(t.x, t.y), make_float2(t.z, t.w)}; }
__device__ __forceinline__ float4 to4(const c2 &a) { return make_float4(a.r.x, a.r.y, a.i.x, a.i.y); }

// a * w and a * conj(w) for one twiddle w given as a broadcast float4 (wr, wr, wi, wi).
__device__ __forceinline__ c2 cmul_b(const c2 &a, float4 w) {
  const float2 wr = make_float2(w.x, w.y), wi = make_float2(w.z, w.w);
  const float2 nwi = pmul(wi, make_float2(-1.f, -1.f));
  return {pfma(a.i, nwi, pmul(a.r, wr)), pfma(a.i, wr, pmul(a.r, wi))};
}
__device__ __forceinline__ c2 cmulc_b(const c2 &a, float4 w) {
  const float2 wr = make_float2(w.x, w.y), wi = make_float2(w.z, w.w);
  const float2 nwi = pmul(wi, make_float2(-1.f, -1.f));
  return {pfma(a.i, wi, pmul(a.r, wr)), pfma(a.r, nwi, pmul(a.i, wr))};
}
// product of two broadcast twiddles, still broadcast
__device__ __forceinline__ float4 wmul_b(float4 a, float4 b) {
  const float2 ar = make_float2(a.x, a.y), ai = make_float2(a.z, a.w);
  const float2 br = make_float2(b.x, b.y), bi = make_float2(b.z, b.w);
  const float2 nbi = pmul(bi, make_float2(-1.f, -1.f));
  const float2 r = pfma(ai, nbi, pmul(ar, br)), i = pfma(ai, br, pmul(ar, bi));
  return make_float4(r.x, r.y, i.x, i.y);
}
__device__ __forceinline__ float4 bcast4(float2 w) { return make_float4(w.x, w.x, w.y, w.y); }

// ------------------------------------------------------------------ small DFTs on c2
// y[k] = sum_n x[n] exp(DIR*2*pi*j*n*k/R), natural order in and out.
template <int DIR>
__device__ __forceinline__ void dft2p(c2 &a, c2 &b) {
  const c2 t = a;
  a = cadd2(t, b);
  b = csub2(t, b);
}

// multiply-by-(DIR*j) is folded into the adds: DIR=-1: -j*(tr,ti) = (ti,-tr); DIR=+1: (-ti, tr)
template <int DIR>
__device__ __forceinline__ void dft4p(c2 &a0, c2 &a1, c2 &a2, c2 &a3) {
  const c2 s0 = cadd2(a0, a2), d0 = csub2(a0, a2);
  const c2 s1 = cadd2(a1, a3), t = csub2(a1, a3);
  a0 = cadd2(s0, s1);
  a2 = csub2(s0, s1);
  if (DIR < 0) {
    a1 = {padd(d0.r, t.i), psub(d0.i, t.r)};
    a3 = {psub(d0.r, t.i), padd(d0.i, t.r)};
  } else {
    a1 = {psub(d0.r, t.i), padd(d0.i, t.r)};
    a3 = {padd(d0.r, t.i), psub(d0.i, t.r)};
  }
}

template <int DIR>
__device__ __forceinline__ void dft8p(c2 (&x)[8]) {
  const float2 h = bc(0.70710678118654752440f), nh = bc(-0.70710678118654752440f);
  dft4p<DIR>(x[0], x[2], x[4], x[6]);   // even samples -> E0..E3 at x[0],x[2],x[4],x[6]
  dft4p<DIR>(x[1], x[3], x[5], x[7]);   // odd samples  -> O0..O3 at x[1],x[3],x[5],x[7]
  const c2 e0 = x[0], e1 = x[2], e2 = x[4], e3 = x[6];
  const c2 o0 = x[1], o1 = x[3], o2 = x[5], o3 = x[7];
  x[0] = cadd2(e0, o0);
  x[4] = csub2(e0, o0);
  // k = 2: t = DIR*j*o2
  if (DIR < 0) {
    x[2] = {padd(e2.r, o2.i), psub(e2.i, o2.r)};
    x[6] = {psub(e2.r, o2.i), padd(e2.i, o2.r)};
  } else {
    x[2] = {psub(e2.r, o2.i), padd(e2.i, o2.r)};
    x[6] = {padd(e2.r, o2.i), psub(e2.i, o2.r)};
  }
  // k = 1: w = (1 + DIR*j)/sqrt2 ; k = 3: w = (-1 + DIR*j)/sqrt2.  With s = or+oi, d = oi-or:
  //   DIR=-1: o*w8^1 = h*(s, d)       o*w8^3 = h*(d, -s)
  //   DIR=+1: o*w8^1 = h*(-d, s)      o*w8^3 = h*(-s, -d)
  {
    const float2 s = padd(o1.r, o1.i), d = psub(o1.i, o1.r);
    if (DIR < 0) {
      x[1] = {pfma(s, h, e1.r), pfma(d, h, e1.i)};
      x[5] = {pfma(s, nh, e1.r), pfma(d, nh, e1.i)};
    } else {
      x[1] = {pfma(d, nh, e1.r), pfma(s, h, e1.i)};
      x[5] = {pfma(d, h, e1.r), pfma(s, nh, e1.i)};
    }
  }
  {
    const float2 s = padd(o3.r, o3.i), d = psub(o3.i, o3.r);
    if (DIR < 0) {
      x[3] = {pfma(d, h, e3.r), pfma(s, nh, e3.i)};
      x[7] = {pfma(d, nh, e3.r), pfma(s, h, e3.i)};
    } else {
      x[3] = {pfma(s, nh, e3.r), pfma(d, nh, e3.i)};
      x[7] = {pfma(s, h, e3.r), pfma(d, h, e3.i)};
    }
  }
}

// t = o * (c + DIR*j*s), then (e + t, e - t)
template <int DIR>
__device__ __forceinline__ void bfly_w(const c2 &e, const c2 &o, float c, float s, c2 &lo, c2 &hi) {
  const float sg = DIR < 0 ? -1.f : 1.f;
  const float2 wr = bc(c), wi = bc(sg * s), nwi = bc(-sg * s);
  const c2 t = {pfma(o.i, nwi, pmul(o.r, wr)), pfma(o.i, wr, pmul(o.r, wi))};
  lo = cadd2(e, t);
  hi = csub2(e, t);
}

template <int DIR>
__device__ __forceinline__ void dft16p(c2 (&x)[16]) {
  const float c1 = 0.92387953251128675613f, s1 = 0.38268343236508977173f;
  const float h = 0.70710678118654752440f;
  c2 e[8], o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { e[i] = x[2 * i]; o[i] = x[2 * i + 1]; }
  dft8p<DIR>(e);
  dft8p<DIR>(o);
  x[0] = cadd2(e[0], o[0]);
  x[8] = csub2(e[0], o[0]);
  bfly_w<DIR>(e[1], o[1], c1, s1, x[1], x[9]);
  bfly_w<DIR>(e[2], o[2], h, h, x[2], x[10]);
  bfly_w<DIR>(e[3], o[3], s1, c1, x[3], x[11]);
  if (DIR < 0) {
    x[4] = {padd(e[4].r, o[4].i), psub(e[4].i, o[4].r)};
    x[12] = {psub(e[4].r, o[4].i), padd(e[4].i, o[4].r)};
  } else {
    x[4] = {psub(e[4].r, o[4].i), padd(e[4].i, o[4].r)};
    x[12] = {padd(e[4].r, o[4].i), psub(e[4].i, o[4].r)};
  }
  bfly_w<DIR>(e[5], o[5], -s1, c1, x[5], x[13]);
  bfly_w<DIR>(e[6], o[6], -h, h, x[6], x[14]);
  bfly_w<DIR>(e[7], o[7], -c1, s1, x[7], x[15]);
}

template <int R, int DIR>
__device__ __forceinline__ void dftp(c2 (&x)[R]) {
  if constexpr (R == 2) dft2p<DIR>(x[0], x[1]);
  else if constexpr (R == 4) dft4p<DIR>(x[0], x[1], x[2], x[3]);
  else if constexpr (R == 8) dft8p<DIR>(x);
  else dft16p<DIR>(x);
}

// ------------------------------------------------------------------ memory helpers
// barrier of the four compute warps (the scheduler warp never joins it)
__device__ __forceinline__ void bar_compute() { asm volatile("bar.sync 1, 128;\n" ::: "memory"); }

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ int perm_token(int p, int N) {
  const int half = N >> 1;                       // N is even here
  return p < half ? 2 * p : 2 * (N - 1 - p) + 1;
}

// input element pair -> packed float2 (two adjacent channels)
template <typename T> struct Pair;
template <> struct Pair<float> {
  static constexpr int ES = 4;
  __device__ static float2 ld(const char *s) { return *reinterpret_cast<const float2 *>(s); }
};
template <> struct Pair<__half> {
  static constexpr int ES = 2;
  __device__ static float2 ld(const char *s) { return __half22float2(*reinterpret_cast<const __half2 *>(s)); }
};
template <> struct Pair<__nv_bfloat16> {
  static constexpr int ES = 2;
  __device__ static float2 ld(const char *s) {
    const unsigned u = *reinterpret_cast<const unsigned *>(s);
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
  }
};


// ------------------------------------------------------------------ TMA and mbarrier transaction helpers
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;\n" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}\n"
               ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(bytes) : "memory");
}
// Tiled loads into this block's shared memory; completion is counted in bytes on `bar`.  One destination block only.
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            unsigned long long *bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
               ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(reinterpret_cast<unsigned long long>(map)),
                 "r"(c0), "r"(c1), "r"(c2), "r"((unsigned)__cvta_generic_to_shared(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *smem_dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                            unsigned long long *bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
               ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(reinterpret_cast<unsigned long long>(map)),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"((unsigned)__cvta_generic_to_shared(bar)) : "memory");
}

// ------------------------------------------------------------------ tile descriptors
enum { PH_NONE = 0, PH_P1 = 1, PH_P2 = 2, PH_P3 = 3 };
struct Tile {
  int phase;   // PH_*
  int unit;
  int a;       // n2 (pass 1, 3) or k1 pair index x (pass 2)
  int cb;      // column block inside the unit
  int idx;     // tile number inside its (unit, pass)
  int ready;   // the tiles it depends on had finished when thread 0 looked
};

// Stage walk kept by thread 0: tiles are fetched in increasing order, so it only moves forward.
struct Walk { int stage; unsigned start; };

__device__ __forceinline__ int stage_blocks(const Params &P, int s) {
  const int l = P.lag;
  return (s < P.U ? 1 : 0) + ((s >= l && s < P.U + l) ? 1 : 0) + ((s >= 2 * l && s < P.U + 2 * l) ? 1 : 0);
}

__device__ __forceinline__ Tile decode_tile(const Params &P, Walk &w, unsigned t) {
  Tile tl;
  tl.phase = PH_NONE; tl.unit = tl.a = tl.cb = tl.idx = tl.ready = 0;
  if (t >= P.total_tiles) return tl;
  unsigned cnt = (unsigned)(stage_blocks(P, w.stage) * P.TPU);
  while (t >= w.start + cnt) {
    w.start += cnt;
    ++w.stage;
    cnt = (unsigned)(stage_blocks(P, w.stage) * P.TPU);
  }
  const int s = w.stage;
  const int i = (int)(t - w.start);
  int blk = i / P.TPU;
  tl.idx = i - blk * P.TPU;
  // blocks present in stage s, in order: pass 1 of unit s, pass 2 of unit s-lag, pass 3 of unit s-2*lag
  const int l = P.lag;
  if (s >= P.U) ++blk;                                  // no pass-1 block
  if (blk >= 1 && !(s >= l && s < P.U + l)) ++blk;      // no pass-2 block
  if (blk == 0) { tl.phase = PH_P1; tl.unit = s; tl.a = tl.idx / P.ncb1; tl.cb = tl.idx - tl.a * P.ncb1; }
  else if (blk == 1) { tl.phase = PH_P2; tl.unit = s - l; tl.a = tl.idx / P.ncb2; tl.cb = tl.idx - tl.a * P.ncb2; }
  else { tl.phase = PH_P3; tl.unit = s - 2 * l; tl.a = tl.idx / P.ncb1; tl.cb = tl.idx - tl.a * P.ncb1; }
  return tl;
}

// The one completion counter a tile waits for (nullptr: none).  It must reach P.TPU.
__device__ __forceinline__ const unsigned *dep_counter(const Params &P, const Tile &tl) {
  const Sched *sc = P.sched;
  if (tl.phase == PH_P1) return tl.unit >= P.R ? &sc->done3[tl.unit - P.R] : nullptr;   // ring slot read out
  if (tl.phase == PH_P2) return &sc->done1[tl.unit];
  if (tl.phase == PH_P3) return &sc->done2[tl.unit];
  return nullptr;
}

// Bounded wait (thread 0 only).  false: gave up, or another block gave up.
__device__ __forceinline__ bool wait_deps(const Params &P, const Tile &tl) {
  const unsigned *c = dep_counter(P, tl);
  if (c == nullptr) return true;
  for (unsigned it = 0; it < P.spin_limit; ++it) {
    if (ld_acquire(c) >= (unsigned)P.TPU) {
      return true;
    }
    if (ld_acquire(&P.sched->abort_flag) != 0u) return false;
    __nanosleep(100);
  }
  atomicExch(&P.sched->abort_flag, 1u);
  atomicOr(P.status, FC_DEV_FLAG_TIMEOUT);
  return false;
}

__device__ __forceinline__ void signal_done(const Params &P, const Tile &tl) {   // thread 0, after a block barrier
  __threadfence();
  Sched *sc = P.sched;
  unsigned *c = tl.phase == PH_P1 ? &sc->done1[tl.unit] : (tl.phase == PH_P2 ? &sc->done2[tl.unit] : &sc->done3[tl.unit]);
  atomicAdd(c, 1u);
}

__device__ __forceinline__ float2 *slot_base(const Params &P, int unit) {
  return P.ws + (size_t)(unit % P.R) * (size_t)P.N * (size_t)P.UC;
}

// ------------------------------------------------------------------ pass 1
// Tile (unit, n2, cb): DFT over n1 of 2*CPW channels.  Thread (cp = tid % CPW, j = tid / CPW).
template <typename T, int R1B>
struct Pass1 {
  static constexpr int N1 = 16 * R1B, CPW = NT / R1B, IT = 16 / R1B, ES = Pair<T>::ES;
  static constexpr int ROWB = 2 * CPW * ES, CPR = ROWB / 16;   // bytes and 16-byte chunks per input row slice

  // Shared-memory rows of a tile: [K even half][K odd half][V even half][V odd half], N1/2 rows of ROWB
  // bytes each.  Row n1 of the transform input is row n1 of the even half for n1 < N1/2 and row
  // N1-1-n1 of the odd half otherwise (the odd tokens run backwards).
  static constexpr unsigned BOXB = (N1 / 2) * ROWB, TILEB = 4 * BOXB;
  __device__ static int srow(int n1) { return n1 < N1 / 2 ? n1 : N1 / 2 + (N1 - 1 - n1); }
  __device__ static void issue(const Params &P, const TmaMaps &M, const Tile &tl, float4 *buf, unsigned long long *bar) {
    const int N2 = P.N / N1;
    const int gcol = tl.unit * P.UC + tl.cb * 2 * CPW;
    const int head = gcol / P.head_dim, c = gcol - head * P.head_dim;
    const int r_even = 2 * tl.a, r_odd = 2 * (N2 - 1 - tl.a) + 1;
    char *dst = reinterpret_cast<char *>(buf);
    mbar_expect_tx(bar, TILEB);
    tma_load_4d(dst, &M.k, c, head, r_even, 0, bar);
    tma_load_4d(dst + BOXB, &M.k, c, head, r_odd, 0, bar);
    tma_load_4d(dst + 2 * BOXB, &M.v, c, head, r_even, 0, bar);
    tma_load_4d(dst + 3 * BOXB, &M.v, c, head, r_odd, 0, bar);
  }

  __device__ static void compute(const Params &P, const Tile &tl, float4 *buf, const float4 *twb, int ntab,
                                 double (*red)[4], int tid) {
    const int N2 = P.N / N1;
    const int cp = tid % CPW, j = tid / CPW;
    const char *in = reinterpret_cast<const char *>(buf);
    c2 x[16];
    float2 aK = make_float2(0.f, 0.f), aV = make_float2(0.f, 0.f);
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const int row = srow(j + R1B * p);
      x[p].r = Pair<T>::ld(in + row * ROWB + cp * 2 * ES);
      x[p].i = Pair<T>::ld(in + (N1 + row) * ROWB + cp * 2 * ES);
      aK = pfma(x[p].r, x[p].r, aK);
      aV = pfma(x[p].i, x[p].i, aV);
    }
    {
      const double a = warp_sum_d((double)(aK.x + aK.y)), b = warp_sum_d((double)(aV.x + aV.y));
      if ((tid & 31) == 0) { red[0][tid >> 5] = a; red[1][tid >> 5] = b; }
    }
    bar_compute();                         // every thread has its inputs; the buffer becomes the exchange area
    dftp<16, -1>(x);
    const int tstep = ntab / N1;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      if (p > 0) x[p] = cmul_b(x[p], twb[j * p * tstep]);
      buf[(j + R1B * p) * CPW + cp] = to4(x[p]);
    }
    bar_compute();
    float2 *slot = slot_base(P, tl.unit);
    const int col = tl.cb * 2 * CPW + 2 * cp;
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
      c2 y[R1B];
#pragma unroll
      for (int q = 0; q < R1B; ++q) y[q] = from4(buf[(q + R1B * pp) * CPW + cp]);
      dftp<R1B, -1>(y);
#pragma unroll
      for (int q = 0; q < R1B; ++q) {
        const int k1 = pp + 16 * q;
        float4 *dst = reinterpret_cast<float4 *>(slot + ((size_t)k1 * N2 + tl.a) * P.UC + col);
        __stcg(dst, to4(y[q]));
      }
    }
    if (tid == 0) {
      const size_t s = (size_t)tl.unit * P.TPU + tl.idx;
      P.part_tot[2 * s] = red[0][0] + red[0][1] + red[0][2] + red[0][3];
      P.part_tot[2 * s + 1] = red[1][0] + red[1][1] + red[1][2] + red[1][3];
    }
  }
};

// ------------------------------------------------------------------ pass 2
// Tile (unit, x, cb): bins k1a = x and k1b = N1 - x (x = 0: k1 = 0 and k1 = N1/2, each its own
// partner) of 2*CP channels.  Thread (cp = tid % CP, j = (tid / CP) % R2B, hf = tid / (CP*R2B)): consecutive j
// are consecutive rows, so a quarter warp reads 128 contiguous bytes even when a row is 64 bytes.
template <int R2B>
struct Pass2 {
  static constexpr int N2 = 16 * R2B, CP = NT / (2 * R2B), IT = 16 / R2B, NAB = R2B + 16;
  static constexpr int HALF = N2 * CP;

  __device__ static void issue(const Params &P, const TmaMaps &M, const Tile &tl, float4 *buf, float4 *ab, float2 *chf,
                               unsigned long long *bar, int lane) {
    const int N1 = P.N / N2;
    const int k1a = tl.a, k1b = tl.a == 0 ? N1 / 2 : N1 - tl.a;
    if (lane == 0) {
      const int row0 = (tl.unit % P.R) * N1;                 // first k1 row of the unit's ring slot
      const int x0 = 2 * tl.cb * 2 * CP;                     // floats
      fence_proxy_async();                                   // the rows were written through the generic proxy
      mbar_expect_tx(bar, 2u * N2 * CP * (unsigned)sizeof(float4));
      tma_load_3d(buf, &M.ws2, x0, 0, row0 + k1a, bar);
      tma_load_3d(buf + HALF, &M.ws2, x0, 0, row0 + k1b, bar);
    }
    // per-tile twiddle factors: w_N^(k1*n2) = A[j] * B[p] for n2 = j + R2B*p
    const int ms = P.master_len / P.N;
    for (int e = lane; e < 2 * NAB + 2; e += 32) {
      if (e < 2 * NAB) {
        const int hf = e / NAB, r = e - hf * NAB;
        const int k1 = hf ? k1b : k1a;
        const int m = (r < R2B ? k1 * r : k1 * R2B * (r - R2B)) & (P.N - 1);
        ab[hf * NAB + r] = bcast4(__ldg(P.master + (size_t)m * ms));
      } else {
        const int hf = e - 2 * NAB;
        const int k1 = hf ? k1b : k1a;
        chf[hf] = __ldg(P.master + (size_t)k1 * (P.master_len / (2 * P.N)));      // exp(-j*pi*k1/N)
      }
    }
  }

  __device__ static void compute(const Params &P, const Tile &tl, float4 *buf, const float4 *twb, int ntab,
                                 const float2 *t2, const float4 *ab, const float2 *chf, int tid) {
    const int N1 = P.N / N2, N = P.N;
    const int cp = tid % CP, j = (tid / CP) % R2B, hf = tid / (CP * R2B);
    const bool self = tl.a == 0;
    const int k1 = hf ? (self ? N1 / 2 : N1 - tl.a) : tl.a;
    float4 *Sh = buf + hf * HALF;
    const float4 *Sp = buf + (self ? hf : 1 - hf) * HALF;
    const float4 A = ab[hf * NAB + j];
    const float4 *B = ab + hf * NAB + R2B;
    const int tstep = ntab / N2;
    c2 x[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      x[p] = from4(Sh[(j + R2B * p) * CP + cp]);
      x[p] = cmul_b(x[p], wmul_b(A, B[p]));
    }
    dftp<16, -1>(x);
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      if (p > 0) x[p] = cmul_b(x[p], twb[j * p * tstep]);
      Sh[(j + R2B * p) * CP + cp] = to4(x[p]);        // same cell this thread read: no barrier needed before
    }
    bar_compute();
    // second forward stage; registers keep bin k2 = pp + 16*q at index it*R2B + q, shared memory the same
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
      c2 y[R2B];
#pragma unroll
      for (int q = 0; q < R2B; ++q) y[q] = from4(Sh[(q + R2B * pp) * CP + cp]);
      dftp<R2B, -1>(y);
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        x[it * R2B + q] = y[q];
        Sh[(q + R2B * pp) * CP + cp] = to4(y[q]);
      }
    }
    bar_compute();                       // full spectra of both halves are in shared memory
    const float2 ch = chf[hf];
    const float2 half2 = bc(0.5f);
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        const int k2 = pp + 16 * q;
        const int bin = k1 + N1 * k2;
        const bool inL = bin <= P.omega, inH = (N - bin) <= P.omega;
        c2 &Pv = x[it * R2B + q];
        if (bin == 0 || (inL && inH)) {
          Pv.r = make_float2(0.f, 0.f);
          Pv.i = make_float2(0.f, 0.f);
        } else if (inL || inH) {
          const int k2p = (k1 == 0) ? ((N2 - k2) & (N2 - 1)) : (N2 - 1 - k2);
          const c2 Q = from4(Sp[((k2p >> 4) + R2B * (k2p & 15)) * CP + cp]);
          const float2 tt = t2[k2];
          const float sgn = inL ? -0.5f : 0.5f;                  // E = (P -/+ uQ)/2, u = exp(+j*pi*bin/N)
          const float er = ch.x * tt.x - ch.y * tt.y, ei = ch.x * tt.y + ch.y * tt.x;   // exp(-j*pi*bin/N)
          const float2 ur = bc(er * sgn), ui = bc(-ei * sgn), nui = bc(ei * sgn);
          Pv.r = pfma(Q.i, nui, pfma(Q.r, ur, pmul(Pv.r, half2)));
          Pv.i = pfma(Q.i, ur, pfma(Q.r, ui, pmul(Pv.i, half2)));
        }
      }
    }
    // first inverse stage (mirror of the second forward stage), in registers
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      c2 y[R2B];
#pragma unroll
      for (int q = 0; q < R2B; ++q) y[q] = x[it * R2B + q];
      dftp<R2B, +1>(y);
#pragma unroll
      for (int q = 0; q < R2B; ++q) x[it * R2B + q] = y[q];
    }
    bar_compute();                       // all partner reads are done
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
#pragma unroll
      for (int q = 0; q < R2B; ++q) Sh[(q + R2B * pp) * CP + cp] = to4(x[it * R2B + q]);
    }
    bar_compute();
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      x[p] = from4(Sh[(j + R2B * p) * CP + cp]);
      if (p > 0) x[p] = cmulc_b(x[p], twb[j * p * tstep]);
    }
    dftp<16, +1>(x);
    float2 *base = slot_base(P, tl.unit) + (size_t)k1 * N2 * P.UC + tl.cb * 2 * CP + 2 * cp;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const c2 o = cmulc_b(x[p], wmul_b(A, B[p]));
      __stcg(reinterpret_cast<float4 *>(base + (size_t)(j + R2B * p) * P.UC), to4(o));
    }
  }
};

// ------------------------------------------------------------------ pass 3
// Tile (unit, n2, cb): inverse DFT over k1 of 2*CPW channels, |.|^2 summed over them -> one
// partial score per row.  Thread (cp = tid % CPW, j = tid / CPW).
template <int CNT, int S>
struct RowReduce {     // halves the CNT row sums across lanes cp ^ S, then continues with S/2
  __device__ static void run(float (&acc)[16], int cp, int &prow) {
    if constexpr (S >= 1) {
      if constexpr (CNT > 1) {
        constexpr int H = CNT / 2;
        const bool up = (cp & S) != 0;
#pragma unroll
        for (int i = 0; i < H; ++i) {
          const float send = up ? acc[i] : acc[i + H];
          const float keep = up ? acc[i + H] : acc[i];
          acc[i] = keep + __shfl_xor_sync(0xffffffffu, send, S);
        }
        if (up) prow += H;
        RowReduce<H, S / 2>::run(acc, cp, prow);
      } else {
        acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], S);
        RowReduce<1, S / 2>::run(acc, cp, prow);
      }
    }
  }
};

template <int R1B>
struct Pass3 {
  static constexpr int N1 = 16 * R1B, CPW = NT / R1B, IT = 16 / R1B;
  static constexpr int LEFT = CPW >= 16 ? 1 : 16 / CPW;       // row sums a lane ends up with
  static constexpr int DUP = CPW > 16 ? CPW / 16 : 1;         // lanes that end up with the same row sum

  __device__ static void issue(const Params &P, const TmaMaps &M, const Tile &tl, float4 *buf, unsigned long long *bar) {
    mbar_expect_tx(bar, (unsigned)(N1 * CPW * sizeof(float4)));
    tma_load_3d(buf, &M.ws3, 2 * tl.cb * 2 * CPW, tl.a, (tl.unit % P.R) * N1, bar);
  }

  __device__ static void compute(const Params &P, const Tile &tl, float4 *buf, const float4 *twb, int ntab,
                                 double (*red)[4], int tid) {
    const int N2 = P.N / N1;
    const int cp = tid % CPW, j = tid / CPW;
    const int tstep = ntab / N1;
    c2 x[16];
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
      c2 y[R1B];
#pragma unroll
      for (int q = 0; q < R1B; ++q) y[q] = from4(buf[(pp + 16 * q) * CPW + cp]);
      dftp<R1B, +1>(y);
#pragma unroll
      for (int q = 0; q < R1B; ++q) x[it * R1B + q] = y[q];
    }
    bar_compute();                         // all bins read; the buffer becomes the exchange area
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
#pragma unroll
      for (int q = 0; q < R1B; ++q) buf[(q + R1B * pp) * CPW + cp] = to4(x[it * R1B + q]);
    }
    bar_compute();
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      x[p] = from4(buf[(j + R1B * p) * CPW + cp]);
      if (p > 0) x[p] = cmulc_b(x[p], twb[j * p * tstep]);
    }
    dftp<16, +1>(x);
    float acc[16];
    float2 totK = make_float2(0.f, 0.f), totV = make_float2(0.f, 0.f);
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float2 t = pfma(x[p].i, x[p].i, pmul(x[p].r, x[p].r));
      acc[p] = t.x + t.y;
      totK = pfma(x[p].r, x[p].r, totK);
      totV = pfma(x[p].i, x[p].i, totV);
    }
    int prow = 0;
    RowReduce<16, CPW / 2>::run(acc, cp, prow);
    const int gcol = tl.unit * P.UC + tl.cb * 2 * CPW;
    const int head = gcol / P.head_dim, part = (gcol - head * P.head_dim) / (2 * CPW);
    float *dstp = P.nparts > 1 ? P.partial + ((size_t)part * P.num_heads + head) * (size_t)P.N
                               : P.scores + (long long)head * P.score_stride;
    if ((cp & (DUP - 1)) == 0) {
#pragma unroll
      for (int i = 0; i < LEFT; ++i) {
        const int p = (j + R1B * (prow + i)) * N2 + tl.a;
        __stcg(dstp + perm_token(p, P.N), acc[i] * P.inv_scale);
      }
    }
    const double dk = warp_sum_d((double)((totK.x + totK.y) * P.inv_scale));
    const double dv = warp_sum_d((double)((totV.x + totV.y) * P.inv_scale));
    if ((tid & 31) == 0) { red[0][tid >> 5] = dk; red[1][tid >> 5] = dv; }
    bar_compute();                       // partial scores of the tile are issued, warp sums are visible
    if (tid == 0) {
      const size_t s = (size_t)tl.unit * P.TPU + tl.idx;
      P.part_hi[2 * s] = (red[0][0] + red[0][1] + red[0][2] + red[0][3]) * (double)P.head_dim;   // d * sum Dev_k
      P.part_hi[2 * s + 1] = (red[1][0] + red[1][1] + red[1][2] + red[1][3]) * (double)P.head_dim;
    }
  }
};

// ------------------------------------------------------------------ one-column compute variants
// Same tiles, same shared-memory bytes and the same scheduler-side loads as Pass1/2/3, but 256
// compute threads per tile, each owning ONE complex column (K + jV of one channel) and 16 points
// in plain float2 arithmetic: half the registers per thread, twice the resident warps.  The
// intermediate is then ordinary interleaved complex (re, im) per column.  N1 >= 128 only (the
// row sums of pass 3 are reduced inside one warp).
constexpr int NTC1 = 256;
__device__ __forceinline__ void bar_compute1() { asm volatile("bar.sync 1, 256;\n" ::: "memory"); }

template <typename T> struct One;
template <> struct One<float> { __device__ static float ld(const char *s) { return *reinterpret_cast<const float *>(s); } };
template <> struct One<__half> { __device__ static float ld(const char *s) { return __half2float(*reinterpret_cast<const __half *>(s)); } };
template <> struct One<__nv_bfloat16> {
  __device__ static float ld(const char *s) {
    return __uint_as_float((unsigned)(*reinterpret_cast<const unsigned short *>(s)) << 16);
  }
};

template <typename T, int R1B>
struct Pass1S {
  static constexpr int N1 = 16 * R1B, C = NTC1 / R1B, IT = 16 / R1B, ES = Pair<T>::ES, ROWB = C * ES;
  __device__ static void compute(const Params &P, const Tile &tl, float4 *buf4, const float2 *tw, int ntab,
                                 double (*red)[8], int tid) {
    const int N2 = P.N / N1;
    const int c = tid % C, j = tid / C;
    const char *in = reinterpret_cast<const char *>(buf4);
    float2 *S = reinterpret_cast<float2 *>(buf4);
    float2 x[16];
    float aK = 0.f, aV = 0.f;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const int row = Pass1<T, R1B>::srow(j + R1B * p);
      x[p].x = One<T>::ld(in + row * ROWB + c * ES);
      x[p].y = One<T>::ld(in + (N1 + row) * ROWB + c * ES);
      aK = fmaf(x[p].x, x[p].x, aK);
      aV = fmaf(x[p].y, x[p].y, aV);
    }
    {
      const double a = warp_sum_d((double)aK), b = warp_sum_d((double)aV);
      if ((tid & 31) == 0) { red[0][tid >> 5] = a; red[1][tid >> 5] = b; }
    }
    bar_compute1();                        // every thread has its inputs; the buffer becomes the exchange area
    dft_small<16, -1>(x);
    const int tstep = ntab / N1;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      if (p > 0) x[p] = cmul(x[p], tw[j * p * tstep]);
      S[(j + R1B * p) * C + c] = x[p];
    }
    bar_compute1();
    float2 *slot = slot_base(P, tl.unit);
    const int col = tl.cb * C + c;
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
      float2 y[R1B];
#pragma unroll
      for (int q = 0; q < R1B; ++q) y[q] = S[(q + R1B * pp) * C + c];
      dft_small<R1B, -1>(y);
#pragma unroll
      for (int q = 0; q < R1B; ++q) {
        const int k1 = pp + 16 * q;
        __stcg(slot + ((size_t)k1 * N2 + tl.a) * P.UC + col, y[q]);
      }
    }
    if (tid == 0) {
      const size_t s = (size_t)tl.unit * P.TPU + tl.idx;
      double a = 0, b = 0;
#pragma unroll
      for (int w = 0; w < NTC1 / 32; ++w) { a += red[0][w]; b += red[1][w]; }
      P.part_tot[2 * s] = a;
      P.part_tot[2 * s + 1] = b;
    }
  }
};

// Thread (c = tid % C, j = (tid / C) % R2B, hf = tid / (C * R2B)): consecutive j are consecutive
// rows, so a half warp reads 128 contiguous bytes.
template <int R2B>
struct Pass2S {
  static constexpr int N2 = 16 * R2B, C = NTC1 / (2 * R2B), IT = 16 / R2B, NAB = R2B + 16;
  static constexpr int HALF2 = 2 * Pass2<R2B>::HALF;         // float2 per half, as the loads laid it out
  __device__ static void compute(const Params &P, const Tile &tl, float4 *buf4, const float2 *tw, int ntab,
                                 const float2 *t2, const float4 *ab, const float2 *chf, int tid) {
    const int N1 = P.N / N2, N = P.N;
    const int c = tid % C, j = (tid / C) % R2B, hf = tid / (C * R2B);
    const bool self = tl.a == 0;
    const int k1 = hf ? (self ? N1 / 2 : N1 - tl.a) : tl.a;
    float2 *Sh = reinterpret_cast<float2 *>(buf4) + hf * HALF2;
    const float2 *Sp = reinterpret_cast<const float2 *>(buf4) + (self ? hf : 1 - hf) * HALF2;
    const float4 A4 = ab[hf * NAB + j];
    const float2 A = make_float2(A4.x, A4.z);
    const float4 *B = ab + hf * NAB + R2B;
    const int tstep = ntab / N2;
    float2 x[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float4 b4 = B[p];
      x[p] = cmul(Sh[(j + R2B * p) * C + c], cmul(A, make_float2(b4.x, b4.z)));
    }
    dft_small<16, -1>(x);
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      if (p > 0) x[p] = cmul(x[p], tw[j * p * tstep]);
      Sh[(j + R2B * p) * C + c] = x[p];             // same cell this thread read: no barrier needed before
    }
    bar_compute1();
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
      float2 y[R2B];
#pragma unroll
      for (int q = 0; q < R2B; ++q) y[q] = Sh[(q + R2B * pp) * C + c];
      dft_small<R2B, -1>(y);
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        x[it * R2B + q] = y[q];
        Sh[(q + R2B * pp) * C + c] = y[q];
      }
    }
    bar_compute1();                        // full spectra of both halves are in shared memory
    const float2 ch = chf[hf];
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
#pragma unroll
      for (int q = 0; q < R2B; ++q) {
        const int k2 = pp + 16 * q;
        const int bin = k1 + N1 * k2;
        const bool inL = bin <= P.omega, inH = (N - bin) <= P.omega;
        float2 &Pv = x[it * R2B + q];
        if (bin == 0 || (inL && inH)) {
          Pv = make_float2(0.f, 0.f);
        } else if (inL || inH) {
          const int k2p = (k1 == 0) ? ((N2 - k2) & (N2 - 1)) : (N2 - 1 - k2);
          const float2 Q = Sp[((k2p >> 4) + R2B * (k2p & 15)) * C + c];
          const float2 e = cmul(ch, t2[k2]);                      // exp(-j*pi*bin/N)
          const float sgn = inL ? -0.5f : 0.5f;                   // E = (P -/+ uQ)/2, u = exp(+j*pi*bin/N)
          const float ur = e.x * sgn, ui = -e.y * sgn;
          Pv = make_float2(fmaf(Q.x, ur, fmaf(-Q.y, ui, 0.5f * Pv.x)), fmaf(Q.x, ui, fmaf(Q.y, ur, 0.5f * Pv.y)));
        }
      }
    }
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      float2 y[R2B];
#pragma unroll
      for (int q = 0; q < R2B; ++q) y[q] = x[it * R2B + q];
      dft_small<R2B, +1>(y);
#pragma unroll
      for (int q = 0; q < R2B; ++q) x[it * R2B + q] = y[q];
    }
    bar_compute1();                        // all partner reads are done
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R2B * it;
#pragma unroll
      for (int q = 0; q < R2B; ++q) Sh[(q + R2B * pp) * C + c] = x[it * R2B + q];
    }
    bar_compute1();
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      x[p] = Sh[(j + R2B * p) * C + c];
      if (p > 0) x[p] = cmul_conj(x[p], tw[j * p * tstep]);
    }
    dft_small<16, +1>(x);
    float2 *base = slot_base(P, tl.unit) + (size_t)k1 * N2 * P.UC + tl.cb * C + c;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float4 b4 = B[p];
      __stcg(base + (size_t)(j + R2B * p) * P.UC, cmul_conj(x[p], cmul(A, make_float2(b4.x, b4.z))));
    }
  }
};

template <int R1B>
struct Pass3S {
  static constexpr int N1 = 16 * R1B, C = NTC1 / R1B, IT = 16 / R1B;
  static constexpr int DUP = C > 16 ? C / 16 : 1;
  __device__ static void compute(const Params &P, const Tile &tl, float4 *buf4, const float2 *tw, int ntab,
                                 double (*red)[8], int tid) {
    const int N2 = P.N / N1;
    const int c = tid % C, j = tid / C;
    const int tstep = ntab / N1;
    float2 *S = reinterpret_cast<float2 *>(buf4);
    float2 x[16];
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
      float2 y[R1B];
#pragma unroll
      for (int q = 0; q < R1B; ++q) y[q] = S[(pp + 16 * q) * C + c];
      dft_small<R1B, +1>(y);
#pragma unroll
      for (int q = 0; q < R1B; ++q) x[it * R1B + q] = y[q];
    }
    bar_compute1();                        // all bins read; the buffer becomes the exchange area
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int pp = j + R1B * it;
#pragma unroll
      for (int q = 0; q < R1B; ++q) S[(q + R1B * pp) * C + c] = x[it * R1B + q];
    }
    bar_compute1();
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      x[p] = S[(j + R1B * p) * C + c];
      if (p > 0) x[p] = cmul_conj(x[p], tw[j * p * tstep]);
    }
    dft_small<16, +1>(x);
    float acc[16];
    float totK = 0.f, totV = 0.f;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float ek = x[p].x * x[p].x, ev = x[p].y * x[p].y;
      acc[p] = ek + ev;
      totK += ek;
      totV += ev;
    }
    int prow = 0;
    RowReduce<16, C / 2>::run(acc, c, prow);
    const int gcol = tl.unit * P.UC + tl.cb * C;
    const int head = gcol / P.head_dim, part = (gcol - head * P.head_dim) / C;
    float *dstp = P.nparts > 1 ? P.partial + ((size_t)part * P.num_heads + head) * (size_t)P.N
                               : P.scores + (long long)head * P.score_stride;
    if ((c & (DUP - 1)) == 0) {
      const int p = (j + R1B * prow) * N2 + tl.a;
      __stcg(dstp + perm_token(p, P.N), acc[0] * P.inv_scale);
    }
    const double dk = warp_sum_d((double)(totK * P.inv_scale));
    const double dv = warp_sum_d((double)(totV * P.inv_scale));
    if ((tid & 31) == 0) { red[0][tid >> 5] = dk; red[1][tid >> 5] = dv; }
    bar_compute1();
    if (tid == 0) {
      const size_t s = (size_t)tl.unit * P.TPU + tl.idx;
      double a = 0, b = 0;
#pragma unroll
      for (int w = 0; w < NTC1 / 32; ++w) { a += red[0][w]; b += red[1][w]; }
      P.part_hi[2 * s] = a * (double)P.head_dim;
      P.part_hi[2 * s + 1] = b * (double)P.head_dim;
    }
  }
};

// ------------------------------------------------------------------ mbarrier helpers
__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}\n"
               ::"r"((unsigned)__cvta_generic_to_shared(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(unsigned long long *bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"((unsigned)__cvta_generic_to_shared(bar)), "r"(parity) : "memory");
  return ok != 0u;
}
// Bounded wait for a phase of an mbarrier.  false: gave up (and said so), or another block gave up.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity, const Params &P) {
  for (unsigned it = 0; it < P.spin_limit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if ((it & 63u) == 63u && ld_acquire(&P.sched->abort_flag) != 0u) return false;
    __nanosleep(32);
  }
  atomicExch(&P.sched->abort_flag, 1u);
  atomicOr(P.status, FC_DEV_FLAG_TIMEOUT);
  return false;
}

// ------------------------------------------------------------------ the kernel
// Block = 4 compute warps + 1 scheduler warp.  The scheduler warp takes tile numbers, waits for
// the tiles they depend on, fills one of two shared-memory buffers with tiled TMA loads and reports
// finished tiles; the compute warps only ever wait for a full buffer.
// ONE = 0: two packed columns per thread, 128 compute threads; ONE = 1: one column per thread, 256.
template <int ONE> struct Threads { static constexpr int compute = ONE ? NTC1 : NT, all = compute + 32; };

template <int R1B, int R2B, int ONE>
struct Smem {
  static constexpr int N1 = 16 * R1B, N2 = 16 * R2B, NTAB = N1 > N2 ? N1 : N2, NAB = R2B + 16;
  static constexpr size_t tw_bytes = NTAB * (ONE ? sizeof(float2) : sizeof(float4));
  static constexpr size_t bytes = (size_t)2 * BUF4 * sizeof(float4) + tw_bytes + N2 * sizeof(float2) +
                                  2 * 2 * NAB * sizeof(float4) + 2 * 2 * sizeof(float2);
};

// Scheduler warp: report a finished tile (all 32 lanes call it).
template <int R1B>
__device__ __forceinline__ void report_tile(const Params &P, const Tile &tl, int lane) {
  constexpr int N1 = 16 * R1B, CPW = NT / R1B;
  if (lane == 0) signal_done(P, tl);
  if (tl.phase == PH_P3 && P.nparts > 1) {
    // the block that delivers the last partial score of (head, n2) adds all of them in a fixed order
    const int N2 = P.N / N1;
    const int gcol = tl.unit * P.UC + tl.cb * 2 * CPW;
    const int head = gcol / P.head_dim;
    unsigned old = 0u;
    if (lane == 0) {
      unsigned *c = &P.sched->cnt3[head * N2 + tl.a];
      old = atomicAdd(c, 1u);            // after the fence in signal_done
      if (old + 1u == (unsigned)P.nparts) *c = 0u;
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old + 1u == (unsigned)P.nparts) {
      __threadfence();
      for (int n1 = lane; n1 < N1; n1 += 32) {
        const int tok = perm_token(n1 * N2 + tl.a, P.N);
        float sum = 0.f;
        for (int q = 0; q < P.nparts; ++q) sum += __ldcg(P.partial + ((size_t)q * P.num_heads + head) * (size_t)P.N + tok);
        P.scores[(long long)head * P.score_stride + tok] = sum;
      }
    }
  }
}

#ifndef FC_FUSED_MINB
#define FC_FUSED_MINB 3
#endif
template <typename T, int R1B, int R2B, int ONE>
__global__ void __launch_bounds__(Threads<ONE>::all, FC_FUSED_MINB) k_fused(const __grid_constant__ Params P,
                                                                             const __grid_constant__ TmaMaps M) {
  using SM = Smem<R1B, R2B, ONE>;
  constexpr int NTC = Threads<ONE>::compute, NTH = Threads<ONE>::all;
  using P1 = Pass1<T, R1B>;
  using P2 = Pass2<R2B>;
  using P3 = Pass3<R1B>;
  constexpr int NTAB = SM::NTAB, N2 = SM::N2, NAB = SM::NAB;
  extern __shared__ __align__(1024) float4 smem4[];
  float4 *bufs = smem4;                                           // [2][BUF4], TMA destinations (128-byte aligned)
  float4 *twb = smem4 + 2 * BUF4;                                 // [NTAB] exp(-2*pi*j*i/NTAB): broadcast float4, or float2 (ONE)
  float2 *tw1 = reinterpret_cast<float2 *>(twb);
  float2 *t2 = reinterpret_cast<float2 *>(reinterpret_cast<char *>(twb) + SM::tw_bytes);   // [N2] exp(-j*pi*k2/N2)
  float4 *ab = reinterpret_cast<float4 *>(t2 + N2);               // [2 buffers][2 halves][NAB]
  float2 *chf = reinterpret_cast<float2 *>(ab + 2 * 2 * NAB);     // [2 buffers][2 halves]
  __shared__ Tile desc[2];
  __shared__ unsigned long long full[2], done[2];
  __shared__ double red[2][2][8];          // per buffer: a warp may enter the next tile while thread 0 still adds these up
  __shared__ int s_last;
  __shared__ long long stamp[2];
  const int tid = threadIdx.x, lane = tid & 31;
  Sched *sc = P.sched;

  for (int i = tid; i < NTAB; i += NTH) {
    const float2 w = __ldg(P.master + (size_t)i * (P.master_len / NTAB));
    if (ONE) tw1[i] = w; else twb[i] = bcast4(w);
  }
  for (int i = tid; i < N2; i += NTH) t2[i] = __ldg(P.master + (size_t)i * (P.master_len / (2 * N2)));
  if (tid == 0) {
    mbar_init(&full[0], 33u); mbar_init(&full[1], 33u);     // one per scheduler lane + the one that announces the bytes
    mbar_init(&done[0], (unsigned)NTC); mbar_init(&done[1], (unsigned)NTC);
  }
  __syncthreads();

  if (tid >= NTC) {
    // ------------------------------------------------------------ scheduler warp
    Walk walk = {0, 0u};
    unsigned t_next = 0u;
    if (lane == 0) t_next = atomicAdd(&sc->tile_counter, 1u);
    Tile held[2];
    unsigned held_k[2] = {0u, 0u};
    bool live[2] = {false, false};
    unsigned long long n_tiles = 0, n_late = 0, s_back = 0, s_deps = 0, s_issue = 0;
    bool ok = true;
    unsigned k = 0;
    // reports the tile in buffer bb if the compute warps have finished it (never blocks)
    auto poll_report = [&](int bb) {
      if (live[bb] && mbar_test(&done[bb], (held_k[bb] >> 1) & 1u)) {
        report_tile<R1B>(P, held[bb], lane);
        live[bb] = false;
      }
    };
    for (;; ++k) {
      const int b = (int)(k & 1u);
      const long long q0 = clock64();
      const unsigned t = __shfl_sync(0xffffffffu, t_next, 0);
      const Tile tl = decode_tile(P, walk, t);
      if (tl.phase == PH_NONE) break;
      if (lane == 0) t_next = atomicAdd(&sc->tile_counter, 1u);      // answer is needed one tile from now
      // 1. the tiles this one reads must be finished.  While waiting, keep reporting what the compute
      //    warps finish here: it may be exactly what somebody (even this tile) is waiting for.
      const unsigned *dc = dep_counter(P, tl);
      if (dc != nullptr) {
        unsigned it = 0;
        while (true) {
          unsigned v = lane == 0 ? ld_acquire(dc) : 0u;
          v = __shfl_sync(0xffffffffu, v, 0);
          if (v >= (unsigned)P.TPU) break;
          if (it == 0) ++n_late;
          poll_report(0);
          poll_report(1);
          unsigned stop = 0u;
          if (lane == 0) {
            if (++it > P.spin_limit) { atomicExch(&sc->abort_flag, 1u); atomicOr(P.status, FC_DEV_FLAG_TIMEOUT); stop = 1u; }
            else if ((it & 15u) == 15u && ld_acquire(&sc->abort_flag) != 0u) stop = 1u;
          }
          stop = __shfl_sync(0xffffffffu, stop, 0);
          if (stop) { ok = false; break; }
          __nanosleep(64);
        }
        if (!ok) break;
      }
      const long long q1 = clock64();
      // 2. the buffer must be free: the tile that used it two steps ago is finished (and gets reported)
      if (live[b]) {
        if (!mbar_wait(&done[b], (held_k[b] >> 1) & 1u, P)) { ok = false; break; }
        report_tile<R1B>(P, held[b], lane);
        live[b] = false;
      }
      const long long q2 = clock64();
      // 3. descriptor, per-tile tables, then the tile itself through the TMA unit
      float4 *dst = bufs + b * BUF4;
      if (lane == 0) desc[b] = tl;
      if (tl.phase == PH_P2) {
        P2::issue(P, M, tl, dst, ab + b * 2 * NAB, chf + b * 2, &full[b], lane);
        if (lane == 0) stamp[b] = clock64();
      } else if (lane == 0) {
        fence_proxy_async();               // what the counters vouch for was written through the generic proxy
        if (tl.phase == PH_P1) P1::issue(P, M, tl, dst, &full[b]);
        else P3::issue(P, M, tl, dst, &full[b]);
        stamp[b] = clock64();
      }
      __syncwarp();
      __threadfence_block();
      mbar_arrive(&full[b]);               // one per lane: descriptor and tables are written
      s_deps += (unsigned long long)(q1 - q0);
      s_back += (unsigned long long)(q2 - q1);
      s_issue += (unsigned long long)(clock64() - q2);
      held[b] = tl;
      held_k[b] = k;
      live[b] = true;
      ++n_tiles;
    }
    // drain: older buffer first
    for (int jj = 0; jj < 2; ++jj) {
      const int b = (int)((k + jj) & 1u);
      if (live[b]) {
        if (ok && !mbar_wait(&done[b], (held_k[b] >> 1) & 1u, P)) ok = false;
        if (ok) report_tile<R1B>(P, held[b], lane);
        live[b] = false;
      }
    }
    if (ok) {                              // both buffers are idle: hand the compute warps the end marker
      const int b = (int)(k & 1u);
      if (lane == 0) desc[b].phase = PH_NONE;
      __syncwarp();
      __threadfence_block();
      mbar_arrive(&full[b]);
      if (lane == 0) mbar_arrive(&full[b]);   // stands in for the arrival that announces a tile's bytes
    }
    if (lane == 0) {
      atomicAdd(&sc->stats[0], n_tiles);
      atomicAdd(&sc->stats[1], n_late);
      atomicAdd(&sc->stats2[0], s_back);
      atomicAdd(&sc->stats2[1], s_deps);
      atomicAdd(&sc->stats2[2], s_issue);
    }
  } else {
    // ------------------------------------------------------------ compute warps
    unsigned long long c_wait = 0, c_land = 0, c_ph[4] = {0, 0, 0, 0};
    const long long c_begin = clock64();
    for (unsigned k = 0;; ++k) {
      const int b = (int)(k & 1u);
      const long long c0 = clock64();
      if (!mbar_wait(&full[b], (k >> 1) & 1u, P)) break;
      const Tile tl = desc[b];
      if (tl.phase == PH_NONE) break;
      const long long c1 = clock64();
      { const long long l = c1 - stamp[b]; if (c1 - c0 > 64) c_land += (unsigned long long)(l > 0 ? l : 0); }
      float4 *buf = bufs + b * BUF4;
      if constexpr (ONE) {
        if (tl.phase == PH_P1) Pass1S<T, R1B>::compute(P, tl, buf, tw1, NTAB, red[b], tid);
        else if (tl.phase == PH_P2) Pass2S<R2B>::compute(P, tl, buf, tw1, NTAB, t2, ab + b * 2 * NAB, chf + b * 2, tid);
        else Pass3S<R1B>::compute(P, tl, buf, tw1, NTAB, red[b], tid);
      } else {
        if (tl.phase == PH_P1) P1::compute(P, tl, buf, twb, NTAB, reinterpret_cast<double (*)[4]>(red[b]), tid);
        else if (tl.phase == PH_P2) P2::compute(P, tl, buf, twb, NTAB, t2, ab + b * 2 * NAB, chf + b * 2, tid);
        else P3::compute(P, tl, buf, twb, NTAB, reinterpret_cast<double (*)[4]>(red[b]), tid);
      }
      fence_proxy_async();                 // this thread wrote the buffer; the TMA unit writes it next
      mbar_arrive(&done[b]);               // this thread's part of the tile is stored, the buffer is free
      c_wait += (unsigned long long)(c1 - c0);
      c_ph[tl.phase] += (unsigned long long)(clock64() - c1);
    }
    if (tid == 0) {
      atomicAdd(&sc->stats[3], c_ph[PH_P1]);
      atomicAdd(&sc->stats[4], c_ph[PH_P2]);
      atomicAdd(&sc->stats[5], c_ph[PH_P3]);
      atomicAdd(&sc->stats[6], c_wait);
      atomicAdd(&sc->stats2[3], c_land);
      atomicAdd(&sc->stats[7], (unsigned long long)(clock64() - c_begin));
    }
  }
  __syncthreads();

  // ---- exit: the last block to leave adds up the energy partial sums in a fixed order and
  // returns the scheduler state to all-zero
  if (tid == 0) {
    __threadfence();
    const unsigned old = atomicAdd(&sc->exit_counter, 1u);
    s_last = (old + 1u == gridDim.x) ? 1 : 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  double *redd = reinterpret_cast<double *>(smem4);        // [4][NT]
  const int n_part = P.U * P.TPU;
  double a0 = 0, a1 = 0, b0 = 0, b1 = 0;
  if (tid < NT) {
    for (int i = tid; i < n_part; i += NT) {
      a0 += __ldcg(P.part_tot + 2 * i); a1 += __ldcg(P.part_tot + 2 * i + 1);
      b0 += __ldcg(P.part_hi + 2 * i);  b1 += __ldcg(P.part_hi + 2 * i + 1);
    }
    redd[tid] = b0; redd[NT + tid] = a0; redd[2 * NT + tid] = b1; redd[3 * NT + tid] = a1;
  }
  __syncthreads();
  for (int st = NT / 2; st > 0; st >>= 1) {
    if (tid < st)
      for (int q = 0; q < 4; ++q) redd[q * NT + tid] += redd[q * NT + tid + st];
    __syncthreads();
  }
  if (tid < 4) P.energy[tid] = redd[tid * NT];
  for (int i = tid; i < P.U; i += NTH) { sc->done1[i] = 0u; sc->done2[i] = 0u; sc->done3[i] = 0u; }
  const int ncnt = P.nparts > 1 ? P.num_heads * (P.N / (16 * R1B)) : 0;
  for (int i = tid; i < ncnt; i += NTH) sc->cnt3[i] = 0u;
  if (tid == 0) { sc->tile_counter = 0u; sc->exit_counter = 0u; sc->abort_flag = 0u; }
}

}  // namespace fused
