// Handle life cycle, status reporting and the twiddle table of the FlashCache library.
#include "fc_common.cuh"

#include <mutex>
#include <new>
#include <stdlib.h>

namespace {

// master[i] = exp(-2*pi*j*i/len), evaluated in fp64 and rounded once to fp32.
__global__ void k_fill_master(float2 *master, int len) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= len) return;
  double s, c;
  sincospi(-2.0 * (double)i / (double)len, &s, &c);
  master[i] = make_float2((float)c, (float)s);
}

// FP32 throughput probe: every thread runs eight independent chains of packed fused multiply-adds
// (two fp32 lanes per instruction), 4 x 8 of them per iteration, nothing else in the loop.
__global__ void __launch_bounds__(256) k_fma_probe(float *out, int iters, float a, float b) {
  float2 x[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = make_float2(threadIdx.x * 0.001f + i, threadIdx.x * 0.002f - i);
  const float2 aa = make_float2(a, a), bb = make_float2(b, b);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int i = 0; i < 8; ++i) x[i] = __ffma2_rn(x[i], aa, bb);
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += x[i].x + x[i].y;
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// Self test of the failure path every bounded device-side wait takes: one block waits on a shared-memory
// barrier that nothing ever arrives on, gives up after `limit` tries, records the timeout in the status
// word and returns normally.
__global__ void k_selftest_bounded_wait(int *status, unsigned limit) {
  __shared__ unsigned long long bar;
  const unsigned addr = (unsigned)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(addr) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();
  bool done = false;
  for (unsigned it = 0; it < limit && !done; ++it) {
    unsigned ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], 0;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(addr) : "memory");
    done = ok != 0;
  }
  if (!done && threadIdx.x == 0) atomicOr(status, FC_DEV_FLAG_TIMEOUT);
}

}  // namespace

// The persisting part of L2 is a setting of the whole context.  The handles of a device share one claim:
// the first handle that needs it raises the limit (never lowers what the application had set), the last one
// to let go puts the application's value back.  Lines are never reset: only the handle's own stream windows
// are cleared, so another user of persisting L2 in the process keeps what it has.
namespace {
constexpr int kMaxPersistDevices = 64;
std::mutex g_persist_mutex;
int g_persist_claims[kMaxPersistDevices];
size_t g_persist_prev[kMaxPersistDevices];
}  // namespace

bool fc_persist_acquire(fc_handle *h) {
  if (h->persist_on) return true;
  if (h->device < 0 || h->device >= kMaxPersistDevices) return false;
  std::lock_guard<std::mutex> lock(g_persist_mutex);
  if (g_persist_claims[h->device] == 0) {
    size_t prev = 0;
    if (cudaDeviceGetLimit(&prev, cudaLimitPersistingL2CacheSize) != cudaSuccess) { cudaGetLastError(); return false; }
    if (prev < h->persist_max &&
        cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, h->persist_max) != cudaSuccess) { cudaGetLastError(); return false; }
    g_persist_prev[h->device] = prev;
  }
  g_persist_claims[h->device]++;
  h->persist_on = 1;
  return true;
}

void fc_persist_release(fc_handle *h) {
  if (!h->persist_on) return;
  for (int i = 0; i < FC_MAX_AUX; ++i) {
    if (h->aux[i] && h->window_base[i]) {
      cudaStreamAttrValue av = {};
      av.accessPolicyWindow.num_bytes = 0;
      if (cudaStreamSetAttribute(h->aux[i], cudaStreamAttributeAccessPolicyWindow, &av) != cudaSuccess) cudaGetLastError();
    }
    h->window_base[i] = nullptr;
    h->window_bytes[i] = 0;
  }
  h->persist_on = 0;
  if (h->device < 0 || h->device >= kMaxPersistDevices) return;
  std::lock_guard<std::mutex> lock(g_persist_mutex);
  if (--g_persist_claims[h->device] == 0 && g_persist_prev[h->device] < h->persist_max)
    if (cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, g_persist_prev[h->device]) != cudaSuccess) cudaGetLastError();
}

static bool create_streams(fc_handle *h) {
  for (int i = 0; i < FC_MAX_AUX; ++i) {
    if (cudaStreamCreateWithFlags(&h->aux[i], cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join[i], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_done[0][i], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_done[1][i], cudaEventDisableTiming) != cudaSuccess)
      return false;
  }
  return true;
}

extern "C" fc_status fc_create(fc_handle **out, int device, int32_t max_seqlen) {
  if (!out) return FC_ERR_INVALID_ARG;
  *out = nullptr;
  if (max_seqlen < 1 || max_seqlen > 131072) return FC_ERR_UNSUPPORTED;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return FC_ERR_CUDA;
  FC_CUDA_TRY(cudaSetDevice(device));
  fc_handle *h = new (std::nothrow) fc_handle();
  if (!h) return FC_ERR_INTERNAL;
  h->device = device;
  h->max_seqlen = max_seqlen;
  int p2 = 64;
  while (p2 < max_seqlen) p2 <<= 1;
  h->master_len = 4 * p2;
  h->master = nullptr;
  h->status_word = nullptr;
  h->done_counter = nullptr;
  h->group_bytes = (size_t)32 << 20;
  h->tune_cpw = 32;        // tile widths of the specialised kernels in channel pairs (the measured best)
  h->tune_cp = 8;
  h->launches = 0;
  h->num_aux = 2;
  h->ev_fork = nullptr;
  for (int i = 0; i < FC_MAX_AUX; ++i) { h->aux[i] = nullptr; h->ev_join[i] = nullptr; }
  h->prof_class = FC_K_NONE;
  h->prof_events = nullptr;
  h->prof_cap = 0;
  h->prof_used = 0;
  h->prof_stride = 1;
  h->prof_seen = 0;
  h->generic_only = false;
  h->select_overlap = 0;
  h->score_overlap = 0;
  h->band_form = 1;
  h->step = 0;
  h->last_sig = -1;
  h->pending_join = false;
  for (int a = 0; a < 2; ++a) for (int b = 0; b < FC_MAX_AUX; ++b) h->ev_done[a][b] = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete h; return FC_ERR_CUDA; }
  h->num_sms = prop.multiProcessorCount;
  h->l2_persist = 1;
  h->persist_max = (size_t)prop.persistingL2CacheMaxSize;
  h->window_max = (size_t)prop.accessPolicyMaxWindowSize;
  for (int i = 0; i < FC_MAX_AUX; ++i) { h->window_base[i] = nullptr; h->window_bytes[i] = 0; }
  h->persist_on = 0;
  if (cudaMalloc(&h->master, (size_t)h->master_len * sizeof(float2)) != cudaSuccess ||
      cudaMalloc(&h->status_word, sizeof(int)) != cudaSuccess ||
      cudaMemset(h->status_word, 0, sizeof(int)) != cudaSuccess ||
      cudaMalloc(&h->done_counter, 2 * sizeof(unsigned)) != cudaSuccess ||
      cudaMemset(h->done_counter, 0, 2 * sizeof(unsigned)) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      !create_streams(h)) {
    fc_destroy(h);
    return FC_ERR_CUDA;
  }
  {
    // room for the chirp kernel's spectrum of the longest sequence that is not a power of two (transform
    // length: the power of two from 2N-1 up, at most 131072)
    int m = 64;
    const int nmax = max_seqlen < 65536 ? max_seqlen : 65536;
    while (m < 2 * nmax - 1) m <<= 1;
    h->hhat_cache_len = m;
    h->hhat_slot_len = m + 2 * ((nmax + 31) / 32 * 32);
    for (int i = 0; i < FC_HHAT_SLOTS; ++i) h->hhat_cache_n[i] = 0;
    h->hhat_cache_next = 0;
    if (cudaMalloc(&h->hhat_cache, (size_t)FC_HHAT_SLOTS * h->hhat_slot_len * sizeof(float2)) != cudaSuccess) {
      fc_destroy(h);
      return FC_ERR_CUDA;
    }
  }
  k_fill_master<<<(h->master_len + 255) / 256, 256>>>(h->master, h->master_len);
  if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
    fc_destroy(h);
    return FC_ERR_CUDA;
  }
  *out = h;
  return FC_OK;
}

static void free_prof(fc_handle *h) {
  if (h->prof_events) {
    for (int i = 0; i < 2 * h->prof_cap; ++i) cudaEventDestroy(h->prof_events[i]);
    delete[] h->prof_events;
  }
  h->prof_events = nullptr;
  h->prof_cap = h->prof_used = 0;
  h->prof_class = FC_K_NONE;
}

extern "C" fc_status fc_profile_begin(fc_handle *h, int32_t kernel_class, int32_t max_launches) {
  if (!h || kernel_class < FC_K_PASS1 || kernel_class > FC_K_OTHER || max_launches < 1) return FC_ERR_INVALID_ARG;
  free_prof(h);
  h->prof_events = new (std::nothrow) cudaEvent_t[2 * (size_t)max_launches];
  if (!h->prof_events) return FC_ERR_INTERNAL;
  for (int i = 0; i < 2 * max_launches; ++i) {
    if (cudaEventCreate(&h->prof_events[i]) != cudaSuccess) {
      h->prof_cap = i / 2;
      free_prof(h);
      return FC_ERR_CUDA;
    }
  }
  h->prof_cap = max_launches;
  h->prof_used = 0;
  h->prof_seen = 0;
  h->prof_class = kernel_class;
  return FC_OK;
}

extern "C" fc_status fc_profile_stride(fc_handle *h, int32_t stride) {
  if (!h || stride < 1) return FC_ERR_INVALID_ARG;
  h->prof_stride = stride;
  return FC_OK;
}

extern "C" fc_status fc_profile_end(fc_handle *h, double *total_ms, uint64_t *launches) {
  if (!h || !total_ms || !launches) return FC_ERR_INVALID_ARG;
  double sum = 0.0;
  for (int i = 0; i < h->prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(h->prof_events[2 * i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, h->prof_events[2 * i], h->prof_events[2 * i + 1]) != cudaSuccess) {
      free_prof(h);
      return FC_ERR_CUDA;
    }
    sum += (double)ms;
  }
  *total_ms = sum;
  *launches = (uint64_t)h->prof_used;
  free_prof(h);
  return FC_OK;
}

extern "C" void fc_destroy(fc_handle *h) {
  if (!h) return;
  free_prof(h);
  fc_persist_release(h);
  for (int i = 0; i < FC_MAX_AUX; ++i) {
    if (h->aux[i]) cudaStreamSynchronize(h->aux[i]);
    for (int a = 0; a < 2; ++a) if (h->ev_done[a][i]) cudaEventDestroy(h->ev_done[a][i]);
    if (h->aux[i]) cudaStreamDestroy(h->aux[i]);
    if (h->ev_join[i]) cudaEventDestroy(h->ev_join[i]);
  }
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->host_copy) { cudaStreamSynchronize(h->host_copy); cudaStreamDestroy(h->host_copy); }
  for (int i = 0; i < h->host_ev_cap; ++i) cudaEventDestroy(h->host_ev[i]);
  delete[] h->host_ev;
  if (h->ev_inputs_free) cudaEventDestroy(h->ev_inputs_free);
  if (h->ev_outputs_done) cudaEventDestroy(h->ev_outputs_done);
  if (h->hhat_cache) cudaFree(h->hhat_cache);
  if (h->master) cudaFree(h->master);
  if (h->status_word) cudaFree(h->status_word);
  if (h->done_counter) cudaFree(h->done_counter);
  delete h;
}

extern "C" const char *fc_status_string(fc_status s) {
  switch (s) {
    case FC_OK: return "ok";
    case FC_ERR_INVALID_ARG: return "invalid argument";
    case FC_ERR_UNSUPPORTED: return "unsupported dtype, head_dim or sequence length";
    case FC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FC_ERR_CUDA: return "CUDA runtime error";
    case FC_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case FC_ERR_INTERNAL: return "device-side self check failed";
    default: return "unknown status";
  }
}

extern "C" fc_status fc_last_device_status(fc_handle *h, fc_stream stream) {
  if (!h) return FC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    const fc_status fs = fc_flush_pending(h, st);
    if (fs != FC_OK) return fs;
  }
  FC_CUDA_TRY(cudaStreamSynchronize(st));
  int word = 0;
  FC_CUDA_TRY(cudaMemcpy(&word, h->status_word, sizeof(int), cudaMemcpyDeviceToHost));
  if (word != 0) FC_CUDA_TRY(cudaMemset(h->status_word, 0, sizeof(int)));
  if (word == 0) return FC_OK;
  return (word & FC_DEV_FLAG_INTERNAL) ? FC_ERR_INTERNAL : FC_ERR_TIMEOUT;
}

extern "C" fc_status fc_measure_fp32_peak(fc_handle *h, double *tflops) {
  if (!h || !tflops) return FC_ERR_INVALID_ARG;
  FC_CUDA_TRY(cudaSetDevice(h->device));
  const int blocks = h->num_sms * 8, threads = 256, iters = 4000;
  float *out = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  fc_status rc = FC_ERR_CUDA;
  float best_ms = 0.f;
  if (cudaMalloc(&out, (size_t)blocks * threads * sizeof(float)) != cudaSuccess) goto done;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) goto done;
  k_fma_probe<<<blocks, threads>>>(out, 10, 1.0001f, 0.5f);
  for (int rep = 0; rep < 3; ++rep) {
    float ms = 0.f;
    if (cudaEventRecord(e0) != cudaSuccess) goto done;
    k_fma_probe<<<blocks, threads>>>(out, iters, 1.0001f, 0.5f);
    if (cudaEventRecord(e1) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
        cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || cudaGetLastError() != cudaSuccess)
      goto done;
    if (rep == 0 || ms < best_ms) best_ms = ms;
  }
  // flops: 2 per lane and fused multiply-add, 2 lanes per instruction, 32 instructions per iteration
  *tflops = (double)blocks * threads * iters * 32.0 * 2.0 * 2.0 / ((double)best_ms * 1e-3) * 1e-12;
  rc = FC_OK;
done:
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (out) cudaFree(out);
  if (rc != FC_OK) cudaGetLastError();
  return rc;
}

extern "C" fc_status fc_selftest_bounded_wait(fc_handle *h, fc_stream stream) {
  if (!h) return FC_ERR_INVALID_ARG;
  k_selftest_bounded_wait<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(h->status_word, 1000u);
  return fc_after_launch(h);
}

extern "C" uint64_t fc_launch_count(const fc_handle *h) { return h ? (uint64_t)h->launches : 0; }

extern "C" fc_status fc_set_select_overlap(fc_handle *h, int32_t enabled) {
  if (!h) return FC_ERR_INVALID_ARG;
  h->select_overlap = enabled ? 1 : 0;
  return FC_OK;
}

extern "C" fc_status fc_set_score_overlap(fc_handle *h, int32_t enabled) {
  if (!h) return FC_ERR_INVALID_ARG;
  h->score_overlap = enabled ? 1 : 0;
  return FC_OK;
}

extern "C" fc_status fc_set_chirp_band(fc_handle *h, int32_t enabled) {
  if (!h) return FC_ERR_INVALID_ARG;
  h->band_form = enabled ? 1 : 0;
  return FC_OK;
}

extern "C" fc_status fc_set_internal_streams(fc_handle *h, int32_t count) {
  if (!h || count < 1 || count > FC_MAX_AUX) return FC_ERR_INVALID_ARG;
  if (h->pending_join) return FC_ERR_INVALID_ARG;        // work of an earlier call is still on the internal streams
  fc_persist_release(h);                                 // the windows belong to the old set of streams
  h->num_aux = count;
  return FC_OK;
}

extern "C" fc_status fc_set_l2_persist(fc_handle *h, int32_t enabled) {
  if (!h) return FC_ERR_INVALID_ARG;
  h->l2_persist = enabled ? 1 : 0;
  if (!enabled) fc_persist_release(h);
  return FC_OK;
}

extern "C" fc_status fc_reset_ordering(fc_handle *h) {
  if (!h) return FC_ERR_INVALID_ARG;
  h->step = 0;
  h->last_sig = 0;
  h->pending_join = false;
  h->host_last_arena = nullptr;
  for (int i = 0; i < FC_HHAT_SLOTS; ++i) h->hhat_cache_n[i] = 0;
  return FC_OK;
}

extern "C" fc_status fc_set_group_bytes(fc_handle *h, size_t bytes) {
  if (!h || bytes == 0) return FC_ERR_INVALID_ARG;
  h->group_bytes = bytes;
  return FC_OK;
}
