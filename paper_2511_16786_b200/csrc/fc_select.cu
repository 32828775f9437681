// fc_allocate_budgets (Dynamic Budget Allocation Module, Sec. 3.2.2) and
// fc_select_compact (keep the Outlier KVs by budget, Sec. 3.2.1 last sentence):
// fp64 budget arithmetic in one small kernel, an exact radix select per
// (sequence, head) on the fp32 score bits, an ordered compaction of the chosen
// token indices, and a row gather into the dense compacted cache.
//
// This file is compiled with -fmad=false so that the fp64 budget arithmetic is
// the plain IEEE sequence of multiplies, adds and divides it is written as.
#include "fc_common.cuh"

#include <cooperative_groups.h>
#include <math.h>

namespace {

constexpr int kSeqChunk = 64;          // sequences described per launch (kernel-argument table)
struct SeqTable {
  int start[kSeqChunk + 1];            // token offsets of the chunk's sequences (cu_seqlens slice)
};
constexpr int kLayerChunk = 32;        // layers selected by one launch (kernel-argument table)
struct LayerTable {                    // per layer of the chunk: where its scores, rows and outputs live (DEVICE pointers)
  const float *scores[kLayerChunk];
  const char *k[kLayerChunk], *v[kLayerChunk];
  char *out_k[kLayerChunk], *out_v[kLayerChunk];
  int *out_idx[kLayerChunk];
  long long cap[kLayerChunk];          // rows available in the layer's outputs
};

// ---------------------------------------------------------------------------
// budgets
// ---------------------------------------------------------------------------
__device__ double filled_sum(const double *w, int L, double lam, double lo, double hi) {
  double s = 0.0;
  for (int l = 0; l < L; ++l) {
    double q = lam * w[l];
    q = q < lo ? lo : (q > hi ? hi : q);
    s += q;
  }
  return s;
}

// One block per sequence of the chunk.  Shared memory: w[L], cand[2L], fval[2L], frac[L], order[L].
__global__ void __launch_bounds__(256)
k_allocate(const double *__restrict__ energy, int L, int B, int b0, SeqTable st, double rho,
           int min_keep, int *__restrict__ budgets) {
  extern __shared__ double sh[];
  double *w = sh;
  double *cand = w + L;
  double *fval = cand + 2 * L;
  double *frac = fval + 2 * L;
  int *order = reinterpret_cast<int *>(frac + L);
  __shared__ double s_sum;
  __shared__ int s_bad;
  const int tid = threadIdx.x;
  const int b = b0 + blockIdx.x;
  const int N = st.start[blockIdx.x + 1] - st.start[blockIdx.x];
  if (N == 0) {
    for (int l = tid; l < L; l += blockDim.x) budgets[(size_t)l * B + b] = 0;
    return;
  }
  const double lo = (double)(min_keep < N ? (min_keep < 0 ? 0 : min_keep) : N);
  const double hi = (double)N;
  double bt = floor(rho * (double)N * (double)L + 0.5);
  if (bt < (double)L * lo) bt = (double)L * lo;
  if (bt > (double)L * hi) bt = (double)L * hi;
  const long long B_tot = (long long)bt;

  // R^l = hiK/totK + hiV/totV   (Eq. 12)
  if (tid == 0) s_bad = 0;
  __syncthreads();
  for (int l = tid; l < L; l += blockDim.x) {
    const double *e = energy + ((size_t)l * B + b) * 4;
    const double rk = e[1] > 0.0 ? e[0] / e[1] : 0.0;
    const double rv = e[3] > 0.0 ? e[2] / e[3] : 0.0;
    const double R = rk + rv;
    w[l] = R;
    if (!(R >= 0.0) || isinf(R)) s_bad = 1;
  }
  __syncthreads();
  if (tid == 0) {
    double s = 0.0;
    for (int l = 0; l < L; ++l) s += w[l];
    if (!(s > 0.0) || isinf(s) || isnan(s)) s_bad = 1;
    s_sum = s;
  }
  __syncthreads();
  const bool uniform = s_bad != 0;
  const double total = s_sum;
  __syncthreads();
  for (int l = tid; l < L; l += blockDim.x) w[l] = uniform ? 1.0 / (double)L : w[l] / total;
  __syncthreads();

  // kinks of f(lam) = sum clamp(lam*w, lo, hi) and f at each of them
  for (int i = tid; i < 2 * L; i += blockDim.x) {
    const double wl = w[i >> 1];
    cand[i] = wl > 0.0 ? ((i & 1) ? hi / wl : lo / wl) : INFINITY;
  }
  __syncthreads();
  for (int i = tid; i < 2 * L; i += blockDim.x)
    fval[i] = isinf(cand[i]) ? -1.0 : filled_sum(w, L, cand[i], lo, hi);
  __syncthreads();

  if (tid == 0) {
    // smallest kink b* > 0 with f(b*) >= B_tot, and the largest kink a* < b* (0 counts as a kink)
    double bstar = INFINITY, fb = 0.0, kmax = 0.0;
    for (int i = 0; i < 2 * L; ++i) {
      if (isinf(cand[i])) continue;
      if (cand[i] > kmax) kmax = cand[i];
      if (cand[i] > 0.0 && fval[i] >= (double)B_tot && cand[i] < bstar) { bstar = cand[i]; fb = fval[i]; }
    }
    double lam;
    if (isinf(bstar)) {
      lam = kmax;
    } else {
      double astar = 0.0;
      for (int i = 0; i < 2 * L; ++i)
        if (!isinf(cand[i]) && cand[i] < bstar && cand[i] > astar) astar = cand[i];
      const double fa = filled_sum(w, L, astar, lo, hi);
      lam = (fb == fa) ? astar : astar + ((double)B_tot - fa) * (bstar - astar) / (fb - fa);
    }
    long long sum = 0;
    for (int l = 0; l < L; ++l) {
      double q = lam * w[l];
      q = q < lo ? lo : (q > hi ? hi : q);
      const double fl = floor(q);
      frac[l] = q - fl;
      budgets[(size_t)l * B + b] = (int)fl;
      sum += (long long)fl;
    }
    s_sum = (double)(B_tot - sum);     // deficit
  }
  __syncthreads();
  // order by (fraction descending, layer ascending)
  for (int l = tid; l < L; l += blockDim.x) {
    int rank = 0;
    const double f = frac[l];
    for (int m = 0; m < L; ++m) rank += (frac[m] > f || (frac[m] == f && m < l)) ? 1 : 0;
    order[rank] = l;
  }
  __syncthreads();
  if (tid == 0) {
    long long deficit = (long long)s_sum;
    while (deficit > 0) {
      bool gave = false;
      for (int r = 0; r < L && deficit > 0; ++r) {
        int *bl = &budgets[(size_t)order[r] * B + b];
        if (*bl < N) { *bl += 1; --deficit; gave = true; }
      }
      if (!gave) break;
    }
  }
}

__global__ void k_offsets(const int *__restrict__ budgets, int L, int B, long long *__restrict__ out_offsets) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= L) return;
  long long acc = 0;
  out_offsets[(size_t)l * (B + 1)] = 0;
  for (int b = 0; b < B; ++b) {
    acc += budgets[(size_t)l * B + b];
    out_offsets[(size_t)l * (B + 1) + b + 1] = acc;
  }
}

// ---------------------------------------------------------------------------
// selection
// ---------------------------------------------------------------------------
// Monotone map float -> uint32: larger score, larger key.  NaN ranks with +inf, -0 with +0.
__device__ __forceinline__ unsigned score_key(float x) {
  if (x != x) return 0xFF800000u;
  if (x == 0.f) return 0x80000000u;
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 1024;   // threads per block of the selection kernel
constexpr int kSelCluster = 8;      // blocks (one cluster) per (sequence, head) at most; 2 or 4 for shorter sequences
constexpr int kSelKptMax = 16;      // scores per thread: 8 * 1024 * 16 = 131072 tokens at most

// Selection + compaction + row gather for one (sequence, head), by one cluster of
// CL blocks (2, 4 or 8).  Block r of the cluster owns the contiguous token range
// [r*chunk, (r+1)*chunk) and keeps its score keys in registers.  The k-th largest
// key is found by a 4-pass MSB-first radix select whose 256-bin histograms are
// summed across the cluster through distributed shared memory; the chosen tokens
// are then ranked in token order (block prefix + cluster prefix), written as
// ascending indices, and their K/V rows are copied by the same block.
// grid (CL * sequences in chunk, heads), cluster (CL, 1, 1).
// PER_LAYER: one cluster per sequence (grid.y = 1) ranks the tokens by the sum over heads of their
// scores (the order of the head-averaged deviation), writes the same indices for every head and
// gathers the rows of all heads.  protect (may be null): a non-zero byte per token of the batch puts
// that token before every unmarked one.
template <int kSelKpt, bool PER_LAYER, int CL>
__device__ __forceinline__ void
select_gather_body(const float *__restrict__ scores, long long T, const SeqTable &st, int b0,
                const int *__restrict__ budgets, const long long *__restrict__ out_offsets,
                int *__restrict__ out_idx, long long cap, int *__restrict__ status,
                const char *__restrict__ kin, const char *__restrict__ vin, long long stride_token_b,
                long long stride_head_b, int row_bytes, int H, char *__restrict__ out_k,
                char *__restrict__ out_v, const unsigned char *__restrict__ protect) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ int lhist[4][256];          // this block's histograms, one per pass (read by the whole cluster)
  __shared__ int ghist[256];             // cluster-wide histogram of the current pass
  __shared__ unsigned tot[CL];  // (ties << 16 | greater) of every block of the cluster
  __shared__ unsigned wsum[kSelThreads / 32];
  __shared__ unsigned s_prefix;
  __shared__ int s_krem;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned r = cluster.block_rank();
  const int bl = blockIdx.x / CL;
  const int b = b0 + bl, h = PER_LAYER ? 0 : blockIdx.y;
  const int s0 = st.start[bl];
  const int n = st.start[bl + 1] - s0;
  int k = budgets[b];
  k = k < 0 ? 0 : (k > n ? n : k);
  const long long off = out_offsets[b];
  if (k == 0) return;                                    // same decision in every block of the cluster
  if (off < 0 || off + k > cap) {
    if (tid == 0 && r == 0) atomicOr(status, FC_DEV_FLAG_INTERNAL);
    return;
  }
  const float *sc = scores + (long long)h * T + s0;
  int *dst = out_idx + (long long)h * cap + off;

  const int chunk = (n + CL - 1) / CL;
  const int lo = (int)r * chunk;
  const int hi = lo + chunk < n ? lo + chunk : n;
  const int base = lo + tid * kSelKpt;
  int nv = hi - base;
  nv = nv < 0 ? 0 : (nv > kSelKpt ? kSelKpt : nv);
  unsigned key[kSelKpt];
#pragma unroll
  for (int i = 0; i < kSelKpt; ++i) {
    key[i] = 0u;
    if (i < nv) {
      float x = sc[base + i];
      if (PER_LAYER)
        for (int hh = 1; hh < H; ++hh) x += sc[(long long)hh * T + base + i];
      key[i] = (protect && protect[s0 + base + i]) ? 0xFFFFFFFFu : score_key(x);
    }
  }

  for (int i = tid; i < 4 * 256; i += kSelThreads) (&lhist[0][0])[i] = 0;
  unsigned tau = 0;
  int need = 0;
  const bool take_all = (k == n);
  if (!take_all) {
    __syncthreads();                                     // the local histograms are zero
    unsigned prefix = 0, mask = 0;
    int krem = k;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
#pragma unroll
      for (int i = 0; i < kSelKpt; ++i) {
        const bool m = (i < nv) && ((key[i] & mask) == prefix);
        const unsigned act = __ballot_sync(0xffffffffu, m);
        if (m) {
          const unsigned dgt = (key[i] >> shift) & 255u;
          const unsigned peers = __match_any_sync(act, dgt);
          if (lane == __ffs(peers) - 1) atomicAdd(&lhist[pass][dgt], __popc(peers));
        }
      }
      cluster.sync();                                    // every block's histogram of this pass is complete
      if (tid < 256) {
        int v = 0;
#pragma unroll
        for (unsigned rr = 0; rr < CL; ++rr) v += *cluster.map_shared_rank(&lhist[pass][tid], rr);
        ghist[tid] = v;
      }
      __syncthreads();
      if (warp == 0) {
        // lane l owns bins 8l..8l+7; find the bin where the count from the top reaches krem
        int mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) mine += ghist[8 * lane + i];
        int above = mine;                                // inclusive suffix sum over lanes >= l
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, above, o);
          if (lane + o < 32) above += t;
        }
        const int strictly_above = above - mine;
        if (strictly_above < krem && krem <= above) {
          int cum = strictly_above, dsel = 8 * lane;
          for (int i = 7; i >= 0; --i) {
            const int c = ghist[8 * lane + i];
            if (cum + c >= krem) { dsel = 8 * lane + i; break; }
            cum += c;
          }
          s_krem = krem - cum;
          s_prefix = prefix | ((unsigned)dsel << shift);
        }
      }
      __syncthreads();
      krem = s_krem;
      prefix = s_prefix;
      mask |= 0xFFu << shift;
    }
    tau = prefix;
    need = krem;
  }

  // per-thread counts, block exclusive scan of (ties << 16 | greater)
  unsigned cnt = 0;
#pragma unroll
  for (int i = 0; i < kSelKpt; ++i)
    if (i < nv) cnt += (key[i] > tau ? 1u : 0u) + (key[i] == tau ? 0x10000u : 0u);
  unsigned incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const unsigned v = wsum[lane];
    unsigned wi = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    wsum[lane] = wi - v;                                 // exclusive prefix of the warp totals
    if (lane == 31) {
#pragma unroll
      for (unsigned rr = 0; rr < CL; ++rr) *cluster.map_shared_rank(&tot[r], rr) = wi;
    }
  }
  cluster.sync();                                        // also orders wsum for the block
  const unsigned excl = wsum[warp] + incl - cnt;
  int gt_before = 0, tie_before = 0, my_gt = 0, my_tie = 0;
#pragma unroll
  for (unsigned rr = 0; rr < CL; ++rr) {
    const unsigned t = tot[rr];
    if (rr < r) { gt_before += (int)(t & 0xFFFFu); tie_before += (int)(t >> 16); }
    if (rr == r) { my_gt = (int)(t & 0xFFFFu); my_tie = (int)(t >> 16); }
  }
  // (a block holds at most 16384 scores, so neither 16-bit field can overflow)
  int g = gt_before + (int)(excl & 0xFFFFu);
  int ti = tie_before + (int)(excl >> 16);
#pragma unroll
  for (int i = 0; i < kSelKpt; ++i) {
    if (i < nv) {
      int pos = -1;
      if (key[i] > tau) {
        pos = g + (ti < need ? ti : need);
        ++g;
      } else if (key[i] == tau) {
        if (ti < need) pos = g + ti;
        ++ti;
      }
      if (pos >= 0) {
        dst[pos] = base + i;
        if (PER_LAYER)
          for (int hh = 1; hh < H; ++hh) dst[(long long)hh * cap + pos] = base + i;
      }
    }
  }
  __syncthreads();                                       // this block's indices are visible to its warps

  // gather the rows this block selected: ranks [first, first + count)
  const int first = gt_before + (tie_before < need ? tie_before : need);
  int tie_take = need - tie_before;
  tie_take = tie_take < 0 ? 0 : (tie_take > my_tie ? my_tie : tie_take);
  const int count = my_gt + tie_take;
  const int n16 = row_bytes >> 4;
  // a warp takes kGatherRows rows at a time: their indices, then their 16-byte pieces, are requested together, so
  // that several independent round trips to DRAM are in flight per warp instead of one after the other
  constexpr int kGatherRows = 4;
  const int per_head = 2 * n16;
  for (int rr0 = warp * kGatherRows; rr0 < count; rr0 += (kSelThreads / 32) * kGatherRows) {
    long long tok[kGatherRows];
#pragma unroll
    for (int g = 0; g < kGatherRows; ++g) {
      const int rr = rr0 + g < count ? rr0 + g : rr0;            // rows past the end repeat the first (not stored)
      tok[g] = (long long)s0 + dst[first + rr];
    }
    for (int w = lane; w < (PER_LAYER ? H * per_head : per_head); w += 32) {
      const int hh = PER_LAYER ? w / per_head : h;
      const int u = PER_LAYER ? w - hh * per_head : w;
      const bool isv = u >= n16;
      const int uu = isv ? u - n16 : u;
      const char *in = (isv ? vin : kin) + (long long)hh * stride_head_b + 16ll * uu;
      char *out = (isv ? out_v : out_k) + 16ll * uu;
      uint4 val[kGatherRows];
#pragma unroll
      for (int g = 0; g < kGatherRows; ++g) val[g] = *reinterpret_cast<const uint4 *>(in + tok[g] * stride_token_b);
#pragma unroll
      for (int g = 0; g < kGatherRows; ++g)
        if (rr0 + g < count)
          *reinterpret_cast<uint4 *>(out + ((off + first + rr0 + g) * H + hh) * (long long)row_bytes) = val[g];
    }
  }
}

// The kernel: grid (CL * sequences in chunk, heads or 1, layers in chunk); blockIdx.z picks the
// layer's pointers from the table and the layer's rows of budgets [L][B] and out_offsets [L][B+1].
// overlap != 0 (launched with the programmatic-serialisation attribute): the next launch in the stream
// may start as soon as every block of this one has begun, and this grid does not finish before its
// predecessor has, so "the last launch is complete" still means "all of them are".
template <int kSelKpt, bool PER_LAYER, int CL>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(kSelThreads)
k_select_gather(const __grid_constant__ LayerTable lt, long long T, const __grid_constant__ SeqTable st, int b0, int B,
                const int *__restrict__ budgets, const long long *__restrict__ out_offsets,
                int *__restrict__ status, long long stride_token_b,
                long long stride_head_b, int row_bytes, int H, int overlap,
                const unsigned char *__restrict__ protect) {
  if (overlap) asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  const int z = blockIdx.z;
  select_gather_body<kSelKpt, PER_LAYER, CL>(lt.scores[z], T, st, b0, budgets + (size_t)z * B,
                                         out_offsets + (size_t)z * (B + 1), lt.out_idx[z], lt.cap[z], status, lt.k[z], lt.v[z],
                                         stride_token_b, stride_head_b, row_bytes, H, lt.out_k[z], lt.out_v[z], protect);
  if (overlap) asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

fc_status check_cu(const int32_t *cu, int batch) {
  if (!cu || batch < 0 || cu[0] != 0) return FC_ERR_INVALID_ARG;
  for (int b = 0; b < batch; ++b)
    if (cu[b + 1] < cu[b]) return FC_ERR_INVALID_ARG;
  return FC_OK;
}

}  // namespace

extern "C" fc_status fc_allocate_budgets(fc_handle *h, const double *energy, int32_t num_layers,
                                         int32_t batch, const int32_t *cu_seqlens_host, double rho,
                                         int32_t min_keep, int32_t *budgets, int64_t *out_offsets,
                                         fc_stream stream) {
  if (!h || !energy || !budgets || !out_offsets) return FC_ERR_INVALID_ARG;
  if (num_layers < 1 || batch < 0 || min_keep < 0) return FC_ERR_INVALID_ARG;
  if (!(rho >= 0.0) || isinf(rho)) return FC_ERR_INVALID_ARG;
  if (num_layers > 1024) return FC_ERR_UNSUPPORTED;
  fc_status s = check_cu(cu_seqlens_host, batch);
  if (s != FC_OK) return s;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((s = fc_flush_pending(h, st)) != FC_OK) return s;    // the energies may still be in flight on the internal streams
  const int L = num_layers;
  const size_t sm = (size_t)(6 * L) * sizeof(double) + (size_t)L * sizeof(int);
  for (int b0 = 0; b0 < batch; b0 += kSeqChunk) {
    const int nseq = batch - b0 < kSeqChunk ? batch - b0 : kSeqChunk;
    SeqTable tab;
    for (int i = 0; i <= nseq; ++i) tab.start[i] = cu_seqlens_host[b0 + i];
    k_allocate<<<nseq, 256, sm, st>>>(energy, L, batch, b0, tab, rho, min_keep, budgets);
    if ((s = fc_after_launch(h)) != FC_OK) return s;
  }
  k_offsets<<<(L + 127) / 128, 128, 0, st>>>(budgets, L, batch, reinterpret_cast<long long *>(out_offsets));
  return fc_after_launch(h);
}

extern "C" size_t fc_select_workspace_bytes(const fc_handle *h, const fc_kv_view *kv) {
  if (!h || !kv) return 0;
  return 256;   // the selection keeps its state on chip; a token amount so callers can treat both phases alike
}

extern "C" fc_status fc_select_compact(fc_handle *h, const fc_kv_view *kv, const float *scores,
                                       const int32_t *budgets, const int64_t *out_offsets,
                                       void *out_k, void *out_v, int32_t *out_idx,
                                       int64_t out_capacity_rows, void *workspace,
                                       size_t workspace_bytes, fc_stream stream) {
  return fc_select_compact_ex(h, kv, scores, budgets, out_offsets, out_k, out_v, out_idx, out_capacity_rows,
                              nullptr, workspace, workspace_bytes, stream);
}

namespace {

// Argument checks shared by the selection entry points (everything but the per-layer pointers).
fc_status check_select_shape(const fc_handle *h, const fc_kv_view *kv, const void *workspace, size_t workspace_bytes) {
  if (!h || !kv) return FC_ERR_INVALID_ARG;
  if (kv->num_heads <= 0 || kv->head_dim <= 0) return FC_ERR_INVALID_ARG;
  if (kv->dtype != FC_F32 && kv->dtype != FC_F16 && kv->dtype != FC_BF16) return FC_ERR_UNSUPPORTED;
  const int es = kv->dtype == FC_F32 ? 4 : 2;
  if ((kv->head_dim * es) % 16) return FC_ERR_UNSUPPORTED;
  fc_status s = check_cu(kv->cu_seqlens, kv->batch);
  if (s != FC_OK) return s;
  for (int b = 0; b < kv->batch; ++b)
    if (kv->cu_seqlens[b + 1] - kv->cu_seqlens[b] > kSelCluster * kSelThreads * kSelKptMax) return FC_ERR_UNSUPPORTED;
  if ((kv->stride_token * es) % 16 || (kv->stride_head * es) % 16) return FC_ERR_INVALID_ARG;
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < fc_select_workspace_bytes(h, kv))
    return FC_ERR_WORKSPACE;
  return FC_OK;
}

// Launches the selection for `nl` (<= kLayerChunk) layers whose pointers are in `lt`; budgets and
// out_offsets point at the first of these layers' rows.
fc_status launch_select(fc_handle *h, cudaStream_t st, const fc_kv_view *kv, const LayerTable &lt, int nl,
                        const int32_t *budgets, const int64_t *out_offsets, bool per_layer,
                        const unsigned char *protect) {
  const int es = kv->dtype == FC_F32 ? 4 : 2;
  const long long T = kv->cu_seqlens[kv->batch];
  fc_status s;
  for (int b0 = 0; b0 < kv->batch; b0 += kSeqChunk) {
    const int nseq = kv->batch - b0 < kSeqChunk ? kv->batch - b0 : kSeqChunk;
    SeqTable tab;
    for (int i = 0; i <= nseq; ++i) tab.start[i] = kv->cu_seqlens[b0 + i];
    int nmax = 0;
    for (int i = 0; i < nseq; ++i) nmax = tab.start[i + 1] - tab.start[i] > nmax ? tab.start[i + 1] - tab.start[i] : nmax;
    // blocks per (sequence, head): the fewest of 2, 4, 8 that hold the longest sequence at 16 scores per thread.
    // Fewer blocks per cluster let more clusters run at once (8 blocks of 1024 threads: 15 clusters on 148 SMs) and
    // the phases of the radix select wait on cluster barriers, not on bandwidth: measured per step, 8 -> 2 blocks,
    // 0.199 -> 0.158 ms at 28 x 4 heads of 32768 tokens, 1.70 -> 1.12 ms at 32 x 32 heads of 16384; one block is
    // 2..9 % slower than two where it would fit.
    int cl = 2;
    while (cl < kSelCluster && nmax > cl * kSelThreads * kSelKptMax) cl *= 2;
    const int per_thread = (nmax + cl * kSelThreads - 1) / (cl * kSelThreads);
    {
      ProfScope ps(h, FC_K_SELECT, st);
#define FC_SEL_LAUNCH(KPT, PL, CLV)                                                                     \
  do {                                                                                                  \
    cudaLaunchConfig_t lc = {};                                                                         \
    lc.gridDim = dim3(CLV * nseq, (PL) ? 1 : kv->num_heads, nl);                                        \
    lc.blockDim = dim3(kSelThreads);                                                                    \
    lc.stream = st;                                                                                     \
    cudaLaunchAttribute at[1];                                                                          \
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                      \
    at[0].val.programmaticStreamSerializationAllowed = 1;                                               \
    lc.attrs = at;                                                                                      \
    lc.numAttrs = h->select_overlap ? 1 : 0;                                                            \
    launch_err = cudaLaunchKernelEx(&lc, k_select_gather<KPT, PL, CLV>, lt, (long long)T, tab, b0, (int)kv->batch, \
        budgets, reinterpret_cast<const long long *>(out_offsets),                                      \
        h->status_word, (long long)(kv->stride_token * es), (long long)(kv->stride_head * es),          \
        (int)(kv->head_dim * es), (int)kv->num_heads, (int)h->select_overlap, protect);                 \
  } while (0)
#define FC_SEL_KPT(PL, CLV)                                                                             \
  do {                                                                                                  \
    if (per_thread <= 2) FC_SEL_LAUNCH(2, PL, CLV);                                                     \
    else if (per_thread <= 4) FC_SEL_LAUNCH(4, PL, CLV);                                                \
    else if (per_thread <= 8) FC_SEL_LAUNCH(8, PL, CLV);                                                \
    else FC_SEL_LAUNCH(16, PL, CLV);                                                                    \
  } while (0)
      cudaError_t launch_err = cudaSuccess;
      if (per_layer) {
        if (cl == 2) FC_SEL_KPT(true, 2); else if (cl == 4) FC_SEL_KPT(true, 4); else FC_SEL_KPT(true, 8);
      } else {
        if (cl == 2) FC_SEL_KPT(false, 2); else if (cl == 4) FC_SEL_KPT(false, 4); else FC_SEL_KPT(false, 8);
      }
      if (launch_err != cudaSuccess) return FC_ERR_CUDA;
#undef FC_SEL_KPT
#undef FC_SEL_LAUNCH
    }
    if ((s = fc_after_launch(h)) != FC_OK) return s;
  }
  return FC_OK;
}

}  // namespace

extern "C" fc_status fc_select_compact_ex(fc_handle *h, const fc_kv_view *kv, const float *scores,
                                          const int32_t *budgets, const int64_t *out_offsets,
                                          void *out_k, void *out_v, int32_t *out_idx,
                                          int64_t out_capacity_rows, const fc_select_options *opt,
                                          void *workspace, size_t workspace_bytes, fc_stream stream) {
  if (!h || !kv || !kv->k || !kv->v || !scores || !budgets || !out_offsets || !out_k || !out_v || !out_idx)
    return FC_ERR_INVALID_ARG;
  if (out_capacity_rows < 0) return FC_ERR_INVALID_ARG;
  fc_status s = check_select_shape(h, kv, workspace, workspace_bytes);
  if (s != FC_OK) return s;
  if (((uintptr_t)kv->k & 15) || ((uintptr_t)kv->v & 15) || ((uintptr_t)out_k & 15) || ((uintptr_t)out_v & 15))
    return FC_ERR_INVALID_ARG;
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((s = fc_flush_pending(h, st)) != FC_OK) return s;
  LayerTable lt = {};
  lt.scores[0] = scores;
  lt.k[0] = static_cast<const char *>(kv->k);
  lt.v[0] = static_cast<const char *>(kv->v);
  lt.out_k[0] = static_cast<char *>(out_k);
  lt.out_v[0] = static_cast<char *>(out_v);
  lt.out_idx[0] = out_idx;
  lt.cap[0] = out_capacity_rows;
  return launch_select(h, st, kv, lt, 1, budgets, out_offsets, opt && opt->per_layer != 0,
                       opt ? static_cast<const unsigned char *>(opt->protect) : nullptr);
}

extern "C" fc_status fc_select_compact_layers(fc_handle *h, const fc_kv_view *shape, const fc_layer_buffers *layers,
                                              int32_t num_layers, const int32_t *budgets, const int64_t *out_offsets,
                                              const fc_select_options *opt,
                                              void *workspace, size_t workspace_bytes, fc_stream stream) {
  if (!h || !shape || !layers || !budgets || !out_offsets || num_layers < 1) return FC_ERR_INVALID_ARG;
  fc_status s = check_select_shape(h, shape, workspace, workspace_bytes);
  if (s != FC_OK) return s;
  for (int l = 0; l < num_layers; ++l) {
    const fc_layer_buffers &b = layers[l];
    if (!b.k || !b.v || !b.scores || !b.out_k || !b.out_v || !b.out_idx || b.out_capacity_rows < 0) return FC_ERR_INVALID_ARG;
    if (((uintptr_t)b.k & 15) || ((uintptr_t)b.v & 15) || ((uintptr_t)b.out_k & 15) || ((uintptr_t)b.out_v & 15))
      return FC_ERR_INVALID_ARG;
  }
  int dev = -1;
  FC_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((s = fc_flush_pending(h, st)) != FC_OK) return s;
  const int B = shape->batch;
  for (int l0 = 0; l0 < num_layers; l0 += kLayerChunk) {
    const int nl = num_layers - l0 < kLayerChunk ? num_layers - l0 : kLayerChunk;
    LayerTable lt = {};
    for (int i = 0; i < nl; ++i) {
      const fc_layer_buffers &b = layers[l0 + i];
      lt.scores[i] = b.scores;
      lt.k[i] = static_cast<const char *>(b.k);
      lt.v[i] = static_cast<const char *>(b.v);
      lt.out_k[i] = static_cast<char *>(b.out_k);
      lt.out_v[i] = static_cast<char *>(b.out_v);
      lt.out_idx[i] = b.out_idx;
      lt.cap[i] = b.out_capacity_rows;
    }
    s = launch_select(h, st, shape, lt, nl, budgets + (size_t)l0 * B, out_offsets + (size_t)l0 * (B + 1),
                      opt && opt->per_layer != 0,
                      opt ? static_cast<const unsigned char *>(opt->protect) : nullptr);
    if (s != FC_OK) return s;
  }
  return FC_OK;
}

extern "C" int64_t fc_layer_capacity_rows(int32_t num_layers, int32_t batch, const int32_t *cu_seqlens,
                                          double rho, int32_t min_keep) {
  if (num_layers < 1 || batch < 0 || !cu_seqlens || min_keep < 0 || !(rho >= 0.0) || isinf(rho)) return -1;
  if (check_cu(cu_seqlens, batch) != FC_OK) return -1;
  long long rows = 0;
  for (int b = 0; b < batch; ++b) {
    const long long N = cu_seqlens[b + 1] - cu_seqlens[b];
    if (N == 0) continue;
    const double lo = (double)(min_keep < N ? min_keep : N), hi = (double)N, L = (double)num_layers;
    double bt = floor(rho * (double)N * L + 0.5);        // B_tot of the sequence, as k_allocate computes it
    if (bt < L * lo) bt = L * lo;
    if (bt > L * hi) bt = L * hi;
    rows += bt < hi ? (long long)bt : N;                  // one layer gets at most N and at most B_tot
  }
  return rows;
}
