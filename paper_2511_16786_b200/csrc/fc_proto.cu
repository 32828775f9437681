// One radix-16 transform stage, three ways, on the same data: the question "do the tensor cores win a stage of the
// token-axis transform (Eq. 6 as a fast transform) at fp32 accuracy?" answered by measurement, not shipped on the
// compression path.
//
//   x, y : DEVICE float2 [16][ncols]; y[k][c] = sum_p x[p][c] * exp(-2*pi*j*p*k/16)
//   variant 0  plain FP32 pipes: a thread owns two columns and a register-resident radix-16 butterfly
//   variant 1  tensor pipe, warp-level m16n8k8 TF32 products with fp32 accumulation: the stage as the real product
//              [Yr; Yi] = [[Fr, -Fi], [Fi, Fr]] [Xr; Xi] (32 x 32 times 32 x 8 columns per warp step), every operand
//              split into a TF32 head and a TF32 tail, three products kept (head*head, head*tail, tail*head): about
//              21 significant bits, the least that keeps the 1e-3 score tolerance of fp32 inputs
//   variant 2  load and store only (what both pay for moving the tile)
// `repeat` > 1 reruns the arithmetic on the registers that many times before the store (the result is then only
// good for timing): it separates arithmetic throughput from the data movement.
#include "fc_common.cuh"

namespace {

__device__ __forceinline__ unsigned to_tf32(float x) {
  unsigned r;
  asm("cvt.rna.tf32.f32 %0, %1;\n" : "=r"(r) : "f"(x));
  return r;
}

__device__ __forceinline__ void mma_tf32(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// entry (row, col) of the 32 x 32 real form of the 16-point DFT matrix
__device__ __forceinline__ float dft_real_form(int row, int col) {
  const int k = row & 15, p = col & 15;
  float s, c;
  sincospif(-(float)((k * p) & 15) / 8.f, &s, &c);        // exp(-2*pi*j*k*p/16) = c + j*s
  const bool rim = row >= 16, cim = col >= 16;
  if (!rim && !cim) return c;      // Yr += Fr * Xr
  if (!rim && cim) return -s;      // Yr -= Fi * Xi
  if (rim && !cim) return s;       // Yi += Fi * Xr
  return c;                        // Yi += Fr * Xi
}

__global__ void __launch_bounds__(256)
k_proto_alu(const float2 *__restrict__ x, float2 *__restrict__ y, int ncols, int repeat) {
  const int pairs = ncols / 2;
  for (int cp = blockIdx.x * blockDim.x + threadIdx.x; cp < pairs; cp += gridDim.x * blockDim.x) {
    float2 a[16], b[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float4 t = *reinterpret_cast<const float4 *>(x + (size_t)p * ncols + 2 * cp);
      a[p] = make_float2(t.x, t.y);
      b[p] = make_float2(t.z, t.w);
    }
    for (int r = 0; r < repeat; ++r) {
      dft_small<16, -1>(a);
      dft_small<16, -1>(b);
      if (r + 1 < repeat) {
#pragma unroll
        for (int p = 0; p < 16; ++p) { a[p].x *= 0.25f; a[p].y *= 0.25f; b[p].x *= 0.25f; b[p].y *= 0.25f; }
      }
    }
#pragma unroll
    for (int p = 0; p < 16; ++p)
      *reinterpret_cast<float4 *>(y + (size_t)p * ncols + 2 * cp) = make_float4(a[p].x, a[p].y, b[p].x, b[p].y);
  }
}

__global__ void __launch_bounds__(256)
k_proto_copy(const float2 *__restrict__ x, float2 *__restrict__ y, int ncols) {
  const int pairs = ncols / 2;
  for (int cp = blockIdx.x * blockDim.x + threadIdx.x; cp < pairs; cp += gridDim.x * blockDim.x) {
#pragma unroll
    for (int p = 0; p < 16; ++p)
      *reinterpret_cast<float4 *>(y + (size_t)p * ncols + 2 * cp) =
          *reinterpret_cast<const float4 *>(x + (size_t)p * ncols + 2 * cp);
  }
}

__global__ void __launch_bounds__(256)
k_proto_tensor(const float2 *__restrict__ x, float2 *__restrict__ y, int ncols, int repeat) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  // A fragments of the constant matrix, head and tail: [m tile][k step][4]
  unsigned ah[2][4][4], al[2][4][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int row = 16 * mt + g + ((i & 1) ? 8 : 0), col = 8 * ks + t + ((i & 2) ? 4 : 0);
        const float v = dft_real_form(row, col);
        ah[mt][ks][i] = to_tf32(v);
        al[mt][ks][i] = to_tf32(v - __uint_as_float(ah[mt][ks][i]));
      }
  const int warps = (gridDim.x * blockDim.x) >> 5, warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  for (int c0 = 8 * warp; c0 < ncols; c0 += 8 * warps) {
    // points t, t+4, t+8, t+12 of column c0 + g: the B fragments of all four k steps
    float2 v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) v[q] = x[(size_t)(t + 4 * q) * ncols + c0 + g];
    float c[2][4];
    for (int r = 0; r < repeat; ++r) {
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) c[mt][0] = c[mt][1] = c[mt][2] = c[mt][3] = 0.f;
      unsigned bh[4][2], bl[4][2];       // k step ks: rows 8ks + t and 8ks + t + 4 of [Xr; Xi]
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float2 s = v[2 * (ks & 1) + i];
          const float val = ks < 2 ? s.x : s.y;
          bh[ks][i] = to_tf32(val);
          bl[ks][i] = to_tf32(val - __uint_as_float(bh[ks][i]));
        }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          mma_tf32(c[mt], al[mt][ks], bh[ks][0], bh[ks][1]);
          mma_tf32(c[mt], ah[mt][ks], bl[ks][0], bl[ks][1]);
          mma_tf32(c[mt], ah[mt][ks], bh[ks][0], bh[ks][1]);
        }
      if (r + 1 < repeat) {              // timing runs: make the next round depend on this one
#pragma unroll
        for (int q = 0; q < 4; ++q) { v[q].x = fmaf(c[0][q], 1e-30f, v[q].x); v[q].y = fmaf(c[1][q], 1e-30f, v[q].y); }
      }
    }
    // c[0]: Yr, c[1]: Yi; rows g and g + 8, columns c0 + 2t and c0 + 2t + 1
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int k = g + 8 * hh;
      *reinterpret_cast<float4 *>(y + (size_t)k * ncols + c0 + 2 * t) =
          make_float4(c[0][2 * hh], c[1][2 * hh], c[0][2 * hh + 1], c[1][2 * hh + 1]);
    }
  }
}

}  // namespace

extern "C" fc_status fc_proto_dft16_stage(fc_handle *h, const void *x, void *y, int32_t ncols, int32_t variant,
                                          int32_t repeat, fc_stream stream) {
  if (!h || !x || !y || ncols < 8 || (ncols & 7) || repeat < 1 || variant < 0 || variant > 2) return FC_ERR_INVALID_ARG;
  if (((uintptr_t)x & 15) || ((uintptr_t)y & 15)) return FC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int blocks = h->num_sms * 4;
  const float2 *xi = static_cast<const float2 *>(x);
  float2 *yo = static_cast<float2 *>(y);
  if (variant == 0) k_proto_alu<<<blocks, 256, 0, st>>>(xi, yo, ncols, repeat);
  else if (variant == 1) k_proto_tensor<<<blocks, 256, 0, st>>>(xi, yo, ncols, repeat);
  else k_proto_copy<<<blocks, 256, 0, st>>>(xi, yo, ncols);
  return fc_after_launch(h);
}
