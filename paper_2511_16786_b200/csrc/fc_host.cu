// fc_compress_host: the compressor driven from host memory (Sec. 3.2, Fig. 2).  Host code
// only: it sequences the library's own entry points around a copy pipeline.
//
//   copy stream :  H2D K_0 V_0 | H2D K_1 V_1 | ...                    (one event per layer)
//   caller's    :  wait ev_0, score 0 | wait ev_1, score 1 | ... | allocate | D2H budgets
//                  -- host waits here once, learns the rows of every layer --
//                  select (all layers, one launch) | (inputs free) | D2H K rows, V rows, indices | (outputs done)
//
// The next job on the same arena starts its H2D copies at "inputs free", so they run while the
// previous job's rows travel back: both directions of the link are busy in steady state.
#include <math.h>
#include <new>

#include "fc_common.cuh"

namespace {

inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

struct Arena {
  size_t off_k, off_v, layer_in_bytes;
  size_t off_scores, off_energy, off_budgets, off_offsets;
  size_t off_out_k, off_out_v, off_out_idx, off_ws, off_protect;
  size_t ws_bytes, total;
  long long T, rows;
  size_t row_bytes;
};

bool job_shape_ok(const fc_host_job *j) {
  if (!j || !j->cu_seqlens) return false;
  if (j->num_layers < 1 || j->num_layers > 1024 || j->num_heads < 1 || j->head_dim < 1 || j->batch < 0) return false;
  if (j->dtype != FC_F32 && j->dtype != FC_F16 && j->dtype != FC_BF16) return false;
  if (j->cu_seqlens[0] != 0) return false;
  for (int b = 0; b < j->batch; ++b)
    if (j->cu_seqlens[b + 1] < j->cu_seqlens[b]) return false;
  return true;
}

fc_kv_view view_of(const fc_host_job *j, const void *k, const void *v) {
  fc_kv_view kv;
  kv.k = k;
  kv.v = v;
  kv.stride_token = (int64_t)j->num_heads * j->head_dim;
  kv.stride_head = j->head_dim;
  kv.dtype = j->dtype;
  kv.num_heads = j->num_heads;
  kv.head_dim = j->head_dim;
  kv.batch = j->batch;
  kv.cu_seqlens = j->cu_seqlens;
  return kv;
}

// Carve-up of the arena; total == 0 when the shape is not one the kernels take.
Arena carve(const fc_handle *h, const fc_host_job *j) {
  Arena a = {};
  const size_t es = j->dtype == FC_F32 ? 4 : 2;
  const int L = j->num_layers, B = j->batch, H = j->num_heads;
  a.T = j->cu_seqlens[B];
  a.rows = fc_compress_host_rows(L, B, j->cu_seqlens, j->rho, j->min_keep);
  a.row_bytes = (size_t)H * j->head_dim * es;
  const long long T1 = a.T > 0 ? a.T : 1, R1 = a.rows > 0 ? a.rows : 1;
  a.layer_in_bytes = up256((size_t)T1 * a.row_bytes);
  // the workspace queries validate the view; any 16-byte-aligned non-null pointer will do for them
  const fc_kv_view probe = view_of(j, reinterpret_cast<const void *>((uintptr_t)256), reinterpret_cast<const void *>((uintptr_t)256));
  const size_t ws_score = fc_score_workspace_bytes(h, &probe);
  const size_t ws_select = fc_select_workspace_bytes(h, &probe);
  if (a.T > 0 && (ws_score == 0 || ws_select == 0)) return a;
  a.ws_bytes = up256(ws_score > ws_select ? ws_score : ws_select);
  size_t off = 0;
  a.off_k = off;       off += (size_t)L * a.layer_in_bytes;
  a.off_v = off;       off += (size_t)L * a.layer_in_bytes;
  a.off_scores = off;  off += up256((size_t)L * H * T1 * sizeof(float));
  a.off_energy = off;  off += up256((size_t)L * (B > 0 ? B : 1) * 4 * sizeof(double));
  a.off_budgets = off; off += up256((size_t)L * (B > 0 ? B : 1) * sizeof(int32_t));
  a.off_offsets = off; off += up256((size_t)L * (B + 1) * sizeof(int64_t));
  a.off_out_k = off;   off += up256((size_t)R1 * a.row_bytes);
  a.off_out_v = off;   off += up256((size_t)R1 * a.row_bytes);
  a.off_out_idx = off; off += up256((size_t)R1 * H * sizeof(int32_t));
  a.off_ws = off;      off += a.ws_bytes > 0 ? a.ws_bytes : 256;
  a.off_protect = off; off += up256((size_t)T1);
  a.total = off;
  return a;
}

fc_status ensure_pipeline(fc_handle *h, int L) {
  if (!h->host_copy) FC_CUDA_TRY(cudaStreamCreateWithFlags(&h->host_copy, cudaStreamNonBlocking));
  if (!h->ev_inputs_free) FC_CUDA_TRY(cudaEventCreateWithFlags(&h->ev_inputs_free, cudaEventDisableTiming));
  if (!h->ev_outputs_done) FC_CUDA_TRY(cudaEventCreateWithFlags(&h->ev_outputs_done, cudaEventDisableTiming));
  if (h->host_ev_cap < L) {
    cudaEvent_t *ev = new (std::nothrow) cudaEvent_t[L];
    if (!ev) return FC_ERR_INTERNAL;
    for (int i = 0; i < h->host_ev_cap; ++i) ev[i] = h->host_ev[i];
    for (int i = h->host_ev_cap; i < L; ++i) {
      if (cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) != cudaSuccess) {
        for (int k = h->host_ev_cap; k < i; ++k) cudaEventDestroy(ev[k]);
        delete[] ev;
        return FC_ERR_CUDA;
      }
    }
    delete[] h->host_ev;
    h->host_ev = ev;
    h->host_ev_cap = L;
  }
  return FC_OK;
}

// Restores the overlap switches of the handle when the call leaves, whichever way.
struct OverlapScope {
  fc_handle *h;
  int sel, sco;
  explicit OverlapScope(fc_handle *h_) : h(h_), sel(h_->select_overlap), sco(h_->score_overlap) {}
  ~OverlapScope() { h->select_overlap = sel; h->score_overlap = sco; }
};

}  // namespace

extern "C" int64_t fc_compress_host_rows(int32_t num_layers, int32_t batch, const int32_t *cu_seqlens,
                                         double rho, int32_t min_keep) {
  if (!cu_seqlens || num_layers < 1 || batch < 0) return 0;
  int64_t rows = 0;
  const double L = (double)num_layers;
  for (int b = 0; b < batch; ++b) {
    const long long N = (long long)cu_seqlens[b + 1] - cu_seqlens[b];
    if (N <= 0) continue;
    const double lo = (double)(min_keep < N ? (min_keep < 0 ? 0 : min_keep) : N);
    double bt = floor(rho * (double)N * L + 0.5);
    if (bt < L * lo) bt = L * lo;
    if (bt > L * (double)N) bt = L * (double)N;
    rows += (int64_t)bt;
  }
  return rows;
}

extern "C" size_t fc_compress_host_arena_bytes(const fc_handle *h, const fc_host_job *job) {
  if (!h || !job_shape_ok(job)) return 0;
  return carve(h, job).total;
}

extern "C" fc_status fc_compress_host(fc_handle *h, const fc_host_job *job, fc_stream stream) {
  if (!h || !job_shape_ok(job)) return FC_ERR_INVALID_ARG;
  if (!job->k_host || !job->v_host || !job->out_k_host || !job->out_v_host || !job->out_idx_host ||
      !job->budgets_host || !job->offsets_host || !job->layer_rows_host)
    return FC_ERR_INVALID_ARG;
  if (!(job->gamma >= 0.0 && job->gamma <= 1.0) || !(job->rho >= 0.0) || job->out_capacity_rows < 0)
    return FC_ERR_INVALID_ARG;
  const int L = job->num_layers, B = job->batch, H = job->num_heads;
  for (int l = 0; l < L; ++l)
    if (!job->k_host[l] || !job->v_host[l]) return FC_ERR_INVALID_ARG;
  FC_CUDA_TRY(cudaSetDevice(h->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  if (job->cu_seqlens[B] == 0) {               // nothing to compress: every count is zero
    for (int i = 0; i < L * B; ++i) job->budgets_host[i] = 0;
    for (int i = 0; i < L * (B + 1); ++i) job->offsets_host[i] = 0;
    for (int l = 0; l <= L; ++l) job->layer_rows_host[l] = 0;
    return FC_OK;
  }
  {
    const fc_kv_view probe = view_of(job, reinterpret_cast<const void *>((uintptr_t)256), reinterpret_cast<const void *>((uintptr_t)256));
    if (fc_score_workspace_bytes(h, &probe) == 0) return FC_ERR_UNSUPPORTED;
  }
  const Arena a = carve(h, job);
  if (a.total == 0) return FC_ERR_UNSUPPORTED;
  if (!job->arena || ((uintptr_t)job->arena & 255) || job->arena_bytes < a.total) return FC_ERR_WORKSPACE;
  if (a.rows > job->out_capacity_rows) return FC_ERR_WORKSPACE;
  fc_status s = ensure_pipeline(h, L);
  if (s != FC_OK) return s;

  char *base = static_cast<char *>(job->arena);
  float *scores = reinterpret_cast<float *>(base + a.off_scores);
  double *energy = reinterpret_cast<double *>(base + a.off_energy);
  int32_t *budgets = reinterpret_cast<int32_t *>(base + a.off_budgets);
  int64_t *offsets = reinterpret_cast<int64_t *>(base + a.off_offsets);
  void *ws = base + a.off_ws;
  const size_t in_bytes = (size_t)a.T * a.row_bytes;

  // the copies may start once whatever read or wrote this arena before is through with it
  const bool same_arena = (h->host_last_arena == job->arena);
  if (same_arena) {
    FC_CUDA_TRY(cudaStreamWaitEvent(h->host_copy, h->ev_inputs_free, 0));
  } else {
    FC_CUDA_TRY(cudaEventRecord(h->ev_inputs_free, st));
    FC_CUDA_TRY(cudaStreamWaitEvent(h->host_copy, h->ev_inputs_free, 0));
  }
  h->host_last_arena = nullptr;                 // set again only when this job got as far as its selection

  unsigned char *protect = nullptr;
  if (job->protect_host) {
    protect = reinterpret_cast<unsigned char *>(base + a.off_protect);
    FC_CUDA_TRY(cudaMemcpyAsync(protect, job->protect_host, (size_t)a.T, cudaMemcpyHostToDevice, h->host_copy));
  }
  const fc_select_options opt = {job->per_layer, protect};

  OverlapScope restore(h);
  h->score_overlap = 1;                         // score x L, then allocate joins the internal streams
  h->select_overlap = 1;                        // select x L back to back, all inputs ready before the first
  for (int l = 0; l < L; ++l) {
    char *kd = base + a.off_k + (size_t)l * a.layer_in_bytes;
    char *vd = base + a.off_v + (size_t)l * a.layer_in_bytes;
    FC_CUDA_TRY(cudaMemcpyAsync(kd, job->k_host[l], in_bytes, cudaMemcpyHostToDevice, h->host_copy));
    FC_CUDA_TRY(cudaMemcpyAsync(vd, job->v_host[l], in_bytes, cudaMemcpyHostToDevice, h->host_copy));
    FC_CUDA_TRY(cudaEventRecord(h->host_ev[l], h->host_copy));
    FC_CUDA_TRY(cudaStreamWaitEvent(st, h->host_ev[l], 0));
    const fc_kv_view kv = view_of(job, kd, vd);
    s = fc_score_layer(h, &kv, job->gamma, scores + (size_t)l * H * a.T, energy + (size_t)l * B * 4, ws,
                       a.ws_bytes, st);
    if (s != FC_OK) return s;
  }
  s = fc_allocate_budgets(h, energy, L, B, job->cu_seqlens, job->rho, job->min_keep, budgets, offsets, st);
  if (s != FC_OK) return s;
  FC_CUDA_TRY(cudaMemcpyAsync(job->budgets_host, budgets, (size_t)L * B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  FC_CUDA_TRY(cudaMemcpyAsync(job->offsets_host, offsets, (size_t)L * (B + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost, st));
  FC_CUDA_TRY(cudaStreamSynchronize(st));

  int64_t rows = 0;
  for (int l = 0; l < L; ++l) {
    job->layer_rows_host[l] = rows;
    const int64_t r = job->offsets_host[(size_t)l * (B + 1) + B];
    if (r < 0) return FC_ERR_INTERNAL;
    rows += r;
  }
  job->layer_rows_host[L] = rows;
  if (rows > a.rows || rows > job->out_capacity_rows) return FC_ERR_WORKSPACE;

  char *ok = base + a.off_out_k, *ov = base + a.off_out_v;
  int32_t *oi = reinterpret_cast<int32_t *>(base + a.off_out_idx);
  // the previous job on this arena may still be copying its rows back (possibly on another stream)
  if (same_arena) FC_CUDA_TRY(cudaStreamWaitEvent(st, h->ev_outputs_done, 0));
  {
    // every layer in one launch (a layer without rows keeps its entry: its budgets are zero, nothing is written)
    fc_layer_buffers *lb = new (std::nothrow) fc_layer_buffers[L];
    if (!lb) return FC_ERR_INTERNAL;
    for (int l = 0; l < L; ++l) {
      const int64_t r0 = job->layer_rows_host[l], r = job->layer_rows_host[l + 1] - r0;
      lb[l].k = base + a.off_k + (size_t)l * a.layer_in_bytes;
      lb[l].v = base + a.off_v + (size_t)l * a.layer_in_bytes;
      lb[l].scores = scores + (size_t)l * H * a.T;
      lb[l].out_k = ok + (size_t)r0 * a.row_bytes;
      lb[l].out_v = ov + (size_t)r0 * a.row_bytes;
      lb[l].out_idx = oi + (size_t)r0 * H;
      lb[l].out_capacity_rows = r;
    }
    const fc_kv_view shape = view_of(job, nullptr, nullptr);
    s = fc_select_compact_layers(h, &shape, lb, L, budgets, offsets, &opt, ws, a.ws_bytes, st);
    delete[] lb;
    if (s != FC_OK) return s;
  }
  FC_CUDA_TRY(cudaEventRecord(h->ev_inputs_free, st));
  h->host_last_arena = job->arena;
  if (rows > 0) {
    FC_CUDA_TRY(cudaMemcpyAsync(job->out_k_host, ok, (size_t)rows * a.row_bytes, cudaMemcpyDeviceToHost, st));
    FC_CUDA_TRY(cudaMemcpyAsync(job->out_v_host, ov, (size_t)rows * a.row_bytes, cudaMemcpyDeviceToHost, st));
    FC_CUDA_TRY(cudaMemcpyAsync(job->out_idx_host, oi, (size_t)rows * H * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  }
  FC_CUDA_TRY(cudaEventRecord(h->ev_outputs_done, st));
  return FC_OK;
}
