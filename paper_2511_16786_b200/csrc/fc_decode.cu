// Decoding step on the compacted cache (Sec. 3.1, Eq. 3-4): Softmax(q K^T / sqrt(d)) V over the rows the
// compressor kept plus the uncompressed tail.  The step reads every K and V row once and is bound by
// that read, so the design is about keeping HBM busy:
//
//  * grid (splits, KV heads, sequences); a block walks its share of the rows in tiles of 64, filled by
//    tiled TMA loads (128-byte swizzle) into a four-stage shared-memory ring behind mbarriers;
//  * all query heads of a KV head (up to 16) are one 16-row operand of m16n8k16 tensor-core products,
//    so a K/V tile is read from shared memory once for the whole group; each of the 4 warps owns 16
//    rows of the tile and keeps its own running maximum, sum and 16 x 128 fp32 output;
//  * the warps' partial results are merged in shared memory, the splits' in a second small kernel.
#include <cuda.h>

#include "fc_common.cuh"

namespace {

constexpr int kD = 128;                 // head_dim
constexpr int kTile = 64;               // rows per tile
constexpr int kWarps = 4;
constexpr int kThreadsD = 32 * kWarps;
constexpr int kBoxBytes = kTile * 128;  // one TMA box: 64 rows x 64 elements of 2 bytes
constexpr int kStageBytes = 4 * kBoxBytes;   // K low/high halves, V low/high halves
// tiles in the shared-memory ring: 4 (one resident block per SM, three tiles in flight) measured best;
// 2 and 3 (three and two blocks per SM) and 5..7 were slower (1.05, 0.98, 0.84..0.91 against 0.82 ms for
// 28 layers of 65536 rows)
constexpr int kStages = 4;
constexpr unsigned kSuspendNs = 2000u;        // a blocking test of an mbarrier sleeps at most about this long
constexpr unsigned kSpinLimit = 1u << 17;    // such tests before a wait gives up (a quarter of a second)

struct DecodeParams {
  const void *q;
  const long long *offsets;
  const int *tail_len;
  float *part_o;        // [batch][q heads][splits][128]
  float2 *part_ml;      // [batch][q heads][splits]: (running maximum in log2 units, sum)
  int *status;
  int H, Hq, G, nsplit, chunk, tail_cap, has_tail;
  float scale_log2;     // log2(e) / sqrt(d)
};

struct DecodeMaps {
  CUtensorMap k, v, tk, tv;
};

__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}\n"
               ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(bytes) : "memory");
}
// One potentially blocking test: the thread sleeps until the phase completes or a hardware time limit passes.
__device__ __forceinline__ bool mbar_try(unsigned long long *bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"((unsigned)__cvta_generic_to_shared(bar)), "r"(parity), "r"(kSuspendNs) : "memory");
  return ok != 0u;
}
// Bounded wait; false = gave up.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity) {
  for (unsigned it = 0; it < kSpinLimit; ++it)
    if (mbar_try(bar, parity)) return true;
  return false;
}
// Tiled loads into this block's shared memory; completion is counted in bytes on `bar`.  One destination block only.
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            unsigned long long *bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
               ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(reinterpret_cast<unsigned long long>(map)),
                 "r"(c0), "r"(c1), "r"(c2), "r"((unsigned)__cvta_generic_to_shared(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                            unsigned long long *bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
               ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(reinterpret_cast<unsigned long long>(map)),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"((unsigned)__cvta_generic_to_shared(bar)) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(unsigned addr, unsigned (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned addr, unsigned (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// D += A (16x16, row) * B (16x8, col), fp32 accumulation.
template <typename T> struct Mma;
template <> struct Mma<__half> {
  __device__ static void run(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  }
  __device__ static unsigned pack(float x, float y) {
    const __half2 h = __floats2half2_rn(x, y);
    return *reinterpret_cast<const unsigned *>(&h);
  }
  __device__ static __half from_float(float x) { return __float2half_rn(x); }
};
template <> struct Mma<__nv_bfloat16> {
  __device__ static void run(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  }
  __device__ static unsigned pack(float x, float y) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<const unsigned *>(&h);
  }
  __device__ static __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

// Byte offset of the 16-byte chunk `chunk` (0..15 over the 128 channels) of row `row` (0..63) inside a K or V
// half-pair as the two swizzled TMA boxes leave it: channels 0..63 in the first box, 64..127 in the second;
// inside a box a row is 128 bytes and chunk j of row r sits at position j ^ (r & 7).
__device__ __forceinline__ unsigned tile_offset(int row, int chunk) {
  return (unsigned)((chunk >> 3) * kBoxBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

constexpr int kMergeStride = kD + 4;    // floats per row of a warp's output in the merge buffer

// One block: KV head h of sequence b, logical rows [split*chunk, (split+1)*chunk).  Logical rows are the kept
// rows, padded to a multiple of the tile, followed by the tail rows, so that every tile lies in one segment.
template <typename T>
__global__ void __launch_bounds__(kThreadsD)
k_decode_partial(const DecodeParams P, const __grid_constant__ DecodeMaps M) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned long long *full = reinterpret_cast<unsigned long long *>(smem + kStages * kStageBytes);
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;

  const long long off0 = P.offsets[b];
  long long nm = P.offsets[b + 1] - off0;
  const int n_main = nm < 0 ? 0 : (int)nm;
  const int n_main_pad = (n_main + kTile - 1) / kTile * kTile;
  int n_tail = P.has_tail ? P.tail_len[b] : 0;
  n_tail = n_tail < 0 ? 0 : (n_tail > P.tail_cap ? P.tail_cap : n_tail);
  const int total = n_tail > 0 ? n_main_pad + n_tail : n_main;
  const int lo = split * P.chunk;
  const int hi = lo + P.chunk < total ? lo + P.chunk : total;
  const int ntiles = lo < hi ? (hi - lo + kTile - 1) / kTile : 0;

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) mbar_init(&full[i], 1u);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();

  // the query heads of this KV head as the 16 x 128 left operand (rows past the group are zero)
  unsigned qf[kD / 16][4];
  {
    const T *qb = static_cast<const T *>(P.q) + ((long long)b * P.Hq + (long long)h * P.G) * kD;
    const bool r0 = g < P.G, r1 = g + 8 < P.G;
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk) {
      const int c = 16 * kk + 2 * t;
      qf[kk][0] = r0 ? *reinterpret_cast<const unsigned *>(qb + g * kD + c) : 0u;
      qf[kk][1] = r1 ? *reinterpret_cast<const unsigned *>(qb + (g + 8) * kD + c) : 0u;
      qf[kk][2] = r0 ? *reinterpret_cast<const unsigned *>(qb + g * kD + c + 8) : 0u;
      qf[kk][3] = r1 ? *reinterpret_cast<const unsigned *>(qb + (g + 8) * kD + c + 8) : 0u;
    }
  }

  auto issue = [&](int ti, int s) {
    const int row0 = lo + ti * kTile;
    unsigned char *dst = smem + s * kStageBytes;
    mbar_expect_tx(&full[s], (unsigned)kStageBytes);
    if (row0 < n_main_pad) {
      const int r = (int)(off0 + row0);
      tma_load_3d(dst, &M.k, 0, h, r, &full[s]);
      tma_load_3d(dst + kBoxBytes, &M.k, 64, h, r, &full[s]);
      tma_load_3d(dst + 2 * kBoxBytes, &M.v, 0, h, r, &full[s]);
      tma_load_3d(dst + 3 * kBoxBytes, &M.v, 64, h, r, &full[s]);
    } else {
      const int r = row0 - n_main_pad;
      tma_load_4d(dst, &M.tk, 0, h, r, b, &full[s]);
      tma_load_4d(dst + kBoxBytes, &M.tk, 64, h, r, b, &full[s]);
      tma_load_4d(dst + 2 * kBoxBytes, &M.tv, 0, h, r, b, &full[s]);
      tma_load_4d(dst + 3 * kBoxBytes, &M.tv, 64, h, r, b, &full[s]);
    }
  };

  float oacc[kD / 8][4];
#pragma unroll
  for (int j = 0; j < kD / 8; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
  const unsigned sbase = (unsigned)__cvta_generic_to_shared(smem);
  bool failed = false;
  int issued = 0, consumed = 0;

  if (tid == 0)
    for (int ti = 0; ti < kStages - 1 && ti < ntiles; ++ti) { issue(ti, ti); issued = ti + 1; }

  for (int ti = 0; ti < ntiles; ++ti) {
    const int s = ti % kStages;
    if (tid == 0 && ti + kStages - 1 < ntiles) {          // into the stage that the barrier below released last time round
      issue(ti + kStages - 1, (ti + kStages - 1) % kStages);
      issued = ti + kStages;
    }
    const bool got = mbar_wait(&full[s], (unsigned)(ti / kStages) & 1u);
    if (__syncthreads_or(got ? 0 : 1)) { failed = true; consumed = ti; break; }
    const int row0 = lo + ti * kTile;
    int valid = (row0 < n_main_pad ? n_main : total) - row0;
    valid = valid > kTile ? kTile : valid;
    const int wrow = 16 * warp;
    if (wrow < valid) {
      const unsigned sb = sbase + (unsigned)(s * kStageBytes);
      float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      const int mi = lane >> 3;
#pragma unroll
      for (int kk = 0; kk < kD / 16; ++kk) {
        unsigned r[4];
        ldmatrix_x4(sb + tile_offset(wrow + (mi >> 1) * 8 + (lane & 7), 2 * kk + (mi & 1)), r);
        Mma<T>::run(sacc[0], qf[kk], r[0], r[1]);
        Mma<T>::run(sacc[1], qf[kk], r[2], r[3]);
      }
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = wrow + 8 * nb + 2 * t + (e & 1);
          const float sv = key < valid ? sacc[nb][e] * P.scale_log2 : -INFINITY;
          sacc[nb][e] = sv;
          mx[e >> 1] = fmaxf(mx[e >> 1], sv);
        }
      float corr[2], ms[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 1));
        mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 2));
        const float mn = fmaxf(m[i], mx[i]);
        ms[i] = (mn == -INFINITY) ? 0.f : mn;
        corr[i] = exp2f(m[i] - ms[i]);
        m[i] = mn;
      }
      float ps[2] = {0.f, 0.f};
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p = exp2f(sacc[nb][e] - ms[e >> 1]);
          sacc[nb][e] = p;
          ps[e >> 1] += p;
        }
      l[0] = l[0] * corr[0] + ps[0];
      l[1] = l[1] * corr[1] + ps[1];
#pragma unroll
      for (int j = 0; j < kD / 8; ++j) {
        oacc[j][0] *= corr[0]; oacc[j][1] *= corr[0];
        oacc[j][2] *= corr[1]; oacc[j][3] *= corr[1];
      }
      // rows at or past `valid` (another sequence's rows, or memory nobody wrote) have probability 0, but
      // 0 x NaN is NaN: their value rows are cleared before the product.  k0 = first of the two rows a
      // fragment register holds (low half k0, high half k0 + 1).
      const int rem = valid - wrow;
      unsigned vm0 = 0xffffffffu, vm1 = 0xffffffffu;
      if (rem < 16) {
        vm0 = (2 * t < rem ? 0x0000ffffu : 0u) | (2 * t + 1 < rem ? 0xffff0000u : 0u);
        vm1 = (2 * t + 8 < rem ? 0x0000ffffu : 0u) | (2 * t + 9 < rem ? 0xffff0000u : 0u);
      }
      unsigned pa[4];
      pa[0] = Mma<T>::pack(sacc[0][0], sacc[0][1]);
      pa[1] = Mma<T>::pack(sacc[0][2], sacc[0][3]);
      pa[2] = Mma<T>::pack(sacc[1][0], sacc[1][1]);
      pa[3] = Mma<T>::pack(sacc[1][2], sacc[1][3]);
#pragma unroll
      for (int jj = 0; jj < kD / 16; ++jj) {
        unsigned r[4];
        ldmatrix_x4_trans(sb + 2 * kBoxBytes + tile_offset(wrow + (mi & 1) * 8 + (lane & 7), 2 * jj + (mi >> 1)), r);
        r[0] &= vm0; r[2] &= vm0;
        r[1] &= vm1; r[3] &= vm1;
        Mma<T>::run(oacc[2 * jj], pa, r[0], r[1]);
        Mma<T>::run(oacc[2 * jj + 1], pa, r[2], r[3]);
      }
    }
    __syncthreads();                       // everyone is through with stage s before it is filled again
  }
  if (failed) {
    // a load did not arrive in time: say so, give the loads still in flight a bounded chance to land
    // (they write this block's shared memory), and report an empty share
    if (tid == 0) {
      atomicOr(P.status, FC_DEV_FLAG_TIMEOUT);
      for (int ti = consumed; ti < issued; ++ti) mbar_wait(&full[ti % kStages], (unsigned)(ti / kStages) & 1u);
    }
    m[0] = m[1] = -INFINITY;
    l[0] = l[1] = 0.f;
#pragma unroll
    for (int j = 0; j < kD / 8; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
    __syncthreads();
  }

  // merge the four warps (each saw a quarter of every tile), then write this split's share
  float *mo = reinterpret_cast<float *>(smem);                          // [warp][16][kMergeStride]
  float2 *mml = reinterpret_cast<float2 *>(mo + kWarps * 16 * kMergeStride);   // [warp][16]
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    l[i] += __shfl_xor_sync(0xffffffffu, l[i], 1);
    l[i] += __shfl_xor_sync(0xffffffffu, l[i], 2);
  }
  {
    float *w0 = mo + ((size_t)warp * 16 + g) * kMergeStride, *w1 = w0 + 8 * kMergeStride;
#pragma unroll
    for (int j = 0; j < kD / 8; ++j) {
      *reinterpret_cast<float2 *>(w0 + 8 * j + 2 * t) = make_float2(oacc[j][0], oacc[j][1]);
      *reinterpret_cast<float2 *>(w1 + 8 * j + 2 * t) = make_float2(oacc[j][2], oacc[j][3]);
    }
    if (t == 0) {
      mml[warp * 16 + g] = make_float2(m[0], l[0]);
      mml[warp * 16 + g + 8] = make_float2(m[1], l[1]);
    }
  }
  __syncthreads();
  for (int r = 0; r < P.G; ++r) {
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, mml[w * 16 + r].x);
    const float msafe = (mm == -INFINITY) ? 0.f : mm;
    float o = 0.f, ll = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float2 v = mml[w * 16 + r];
      const float f = exp2f(v.x - msafe);
      o += mo[((size_t)w * 16 + r) * kMergeStride + tid] * f;
      ll += v.y * f;
    }
    const size_t slot = ((size_t)b * P.Hq + (size_t)h * P.G + r) * P.nsplit + split;
    P.part_o[slot * kD + tid] = o;
    if (tid == 0) P.part_ml[slot] = make_float2(mm, ll);
  }
}

// out[b][j] = sum over splits of their shares, rescaled to the common maximum, divided by the common sum.
template <typename T>
__global__ void __launch_bounds__(kD)
k_decode_combine(const float *__restrict__ part_o, const float2 *__restrict__ part_ml, int nsplit, T *__restrict__ out) {
  const size_t bj = blockIdx.x;
  const int c = threadIdx.x;
  float mm = -INFINITY;
  for (int s = 0; s < nsplit; ++s) mm = fmaxf(mm, part_ml[bj * nsplit + s].x);
  const float msafe = (mm == -INFINITY) ? 0.f : mm;
  float o = 0.f, ll = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float2 v = part_ml[bj * nsplit + s];
    const float f = exp2f(v.x - msafe);
    o += part_o[(bj * nsplit + s) * kD + c] * f;
    ll += v.y * f;
  }
  out[bj * kD + c] = Mma<T>::from_float(ll > 0.f ? o / ll : 0.f);
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tiles of 64 rows x 64 channels of one head, rows 128 bytes wide in shared memory, 128-byte swizzle.
fc_status encode_rows(CUtensorMap *m, CUtensorMapDataType dt, int rank, const void *base, const cuuint64_t *dims,
                      const cuuint64_t *strides_b) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FC_ERR_CUDA;
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)kTile, 1};
  const cuuint32_t ones[4] = {1, 1, 1, 1};
  const CUresult r = fn(m, dt, (cuuint32_t)rank, const_cast<void *>(base), dims, strides_b, box, ones,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FC_OK : FC_ERR_INTERNAL;
}

constexpr size_t kDecodeSmem = (size_t)kStages * kStageBytes + 64 + 1024;   // ring, barriers, slack to align the ring to 1024 bytes

// Resident blocks of k_decode_partial per SM (the launch is sized to one full wave of them).
int decode_blocks_per_sm() {
  static int n = 0;
  if (n == 0) {
    int v = 0;
    if (cudaFuncSetAttribute(k_decode_partial<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecodeSmem) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, k_decode_partial<__half>, kThreadsD, kDecodeSmem) == cudaSuccess && v > 0)
      n = v;
    else
      n = 1;
    cudaGetLastError();
  }
  return n;
}

struct DecodePlan {
  int nsplit, chunk;
  size_t off_ml, total;
};

fc_status check_decode(const fc_handle *h, const fc_decode_args *a) {
  if (!h || !a || !a->q || !a->cache_k || !a->cache_v || !a->offsets) return FC_ERR_INVALID_ARG;
  if (a->batch < 1 || a->num_heads < 1 || a->num_q_heads < 1 || a->cache_rows < 1 || a->max_rows < 0) return FC_ERR_INVALID_ARG;
  if (a->dtype != FC_F16 && a->dtype != FC_BF16) return FC_ERR_UNSUPPORTED;
  if (a->head_dim != kD) return FC_ERR_UNSUPPORTED;
  if (a->num_q_heads % a->num_heads != 0 || a->num_q_heads / a->num_heads > 16) return FC_ERR_UNSUPPORTED;
  if (a->cache_rows > 0x7fffffffll - 2 * kTile || a->max_rows > 0x7fffffffll - 2 * kTile || a->batch > 65535 ||
      a->num_heads > 65535)
    return FC_ERR_UNSUPPORTED;
  if (((uintptr_t)a->q & 15) || ((uintptr_t)a->cache_k & 15) || ((uintptr_t)a->cache_v & 15)) return FC_ERR_INVALID_ARG;
  const bool tail = a->tail_k || a->tail_v || a->tail_len;
  if (tail) {
    if (!a->tail_k || !a->tail_v || !a->tail_len || a->tail_capacity < 1) return FC_ERR_INVALID_ARG;
    if (((uintptr_t)a->tail_k & 15) || ((uintptr_t)a->tail_v & 15)) return FC_ERR_INVALID_ARG;
  }
  return FC_OK;
}

DecodePlan plan_decode(const fc_handle *h, const fc_decode_args *a) {
  DecodePlan p;
  const long long logical = a->max_rows + (a->tail_k ? kTile - 1 : 0);      // the kept rows are padded to a tile before the tail
  long long tiles = (logical + kTile - 1) / kTile;
  if (tiles < 1) tiles = 1;
  const long long groups = (long long)a->batch * a->num_heads;
  long long want = (long long)decode_blocks_per_sm() * h->num_sms / groups;           // one full wave of resident blocks
  if (want < 1) want = 1;
  if (want > tiles) want = tiles;
  const long long per = (tiles + want - 1) / want;
  p.chunk = (int)(per * kTile);
  p.nsplit = (int)((tiles + per - 1) / per);
  const size_t slots = (size_t)a->batch * a->num_q_heads * p.nsplit;
  p.off_ml = (slots * kD * sizeof(float) + 255) & ~(size_t)255;
  p.total = p.off_ml + ((slots * sizeof(float2) + 255) & ~(size_t)255);
  return p;
}

template <typename T>
fc_status launch_decode(fc_handle *h, const fc_decode_args *a, const DecodePlan &pl, void *out, char *ws, cudaStream_t st) {
  const CUtensorMapDataType dt = sizeof(T) == 2 && std::is_same<T, __half>::value ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                                                  : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  DecodeMaps M;
  fc_status s;
  const cuuint64_t row_b = (cuuint64_t)a->num_heads * kD * 2;
  {
    const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)a->num_heads, (cuuint64_t)a->cache_rows};
    const cuuint64_t str[2] = {(cuuint64_t)kD * 2, row_b};
    if ((s = encode_rows(&M.k, dt, 3, a->cache_k, dims, str)) != FC_OK) return s;
    if ((s = encode_rows(&M.v, dt, 3, a->cache_v, dims, str)) != FC_OK) return s;
  }
  if (a->tail_k) {
    const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)a->num_heads, (cuuint64_t)a->tail_capacity, (cuuint64_t)a->batch};
    const cuuint64_t str[3] = {(cuuint64_t)kD * 2, row_b, row_b * (cuuint64_t)a->tail_capacity};
    if ((s = encode_rows(&M.tk, dt, 4, a->tail_k, dims, str)) != FC_OK) return s;
    if ((s = encode_rows(&M.tv, dt, 4, a->tail_v, dims, str)) != FC_OK) return s;
  } else {
    M.tk = M.k;
    M.tv = M.v;
  }
  DecodeParams P;
  P.q = a->q;
  P.offsets = reinterpret_cast<const long long *>(a->offsets);
  P.tail_len = a->tail_len;
  P.part_o = reinterpret_cast<float *>(ws);
  P.part_ml = reinterpret_cast<float2 *>(ws + pl.off_ml);
  P.status = h->status_word;
  P.H = a->num_heads;
  P.Hq = a->num_q_heads;
  P.G = a->num_q_heads / a->num_heads;
  P.nsplit = pl.nsplit;
  P.chunk = pl.chunk;
  P.tail_cap = a->tail_k ? a->tail_capacity : 0;
  P.has_tail = a->tail_k ? 1 : 0;
  P.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kD));
  const size_t sm = kDecodeSmem;
  FC_CUDA_TRY(cudaFuncSetAttribute(k_decode_partial<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm));
  k_decode_partial<T><<<dim3(pl.nsplit, a->num_heads, a->batch), kThreadsD, sm, st>>>(P, M);
  if ((s = fc_after_launch(h)) != FC_OK) return s;
  k_decode_combine<T><<<(unsigned)(a->batch * a->num_q_heads), kD, 0, st>>>(P.part_o, P.part_ml, pl.nsplit,
                                                                              static_cast<T *>(out));
  return fc_after_launch(h);
}

}  // namespace

extern "C" size_t fc_decode_workspace_bytes(const fc_handle *h, const fc_decode_args *a) {
  if (check_decode(h, a) != FC_OK) return 0;
  return plan_decode(h, a).total;
}

extern "C" fc_status fc_decode_attention(fc_handle *h, const fc_decode_args *a, void *out, void *workspace,
                                         size_t workspace_bytes, fc_stream stream) {
  fc_status s = check_decode(h, a);
  if (s != FC_OK) return s;
  if (!out || ((uintptr_t)out & 15)) return FC_ERR_INVALID_ARG;
  const DecodePlan pl = plan_decode(h, a);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < pl.total) return FC_ERR_WORKSPACE;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((s = fc_flush_pending(h, st)) != FC_OK) return s;
  if (a->dtype == FC_F16) return launch_decode<__half>(h, a, pl, out, static_cast<char *>(workspace), st);
  return launch_decode<__nv_bfloat16>(h, a, pl, out, static_cast<char *>(workspace), st);
}
