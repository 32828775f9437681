/*
 * flashcache.h -- C ABI of the B200 FlashCache compression path.
 *
 * The library runs the prefill-time KV-cache compressor of "Revisiting
 * Multimodal KV Cache Compression: A Frequency-Domain-Guided
 * Outlier-KV-Aware Approach" (FlashCache) on one GPU:
 *
 *     fc_score_layer      x L   Outlier KV Recognition Module   (Sec. 3.2.1, Eq. 5-10)
 *                               + the energy sums of Eq. 11-12  (Sec. 3.2.2)
 *     fc_allocate_budgets x 1   Dynamic Budget Allocation       (Sec. 3.2.2, last paragraph)
 *     fc_select_compact   x L   keep the Outlier KVs by budget  (Sec. 3.2.1, last sentence)
 *
 * Conventions
 *   - Every pointer is marked HOST or DEVICE.  The caller owns every buffer;
 *     the library allocates device memory only in fc_create (and, for its host
 *     pipeline, two streams and a few events on the first fc_compress_host call)
 *     and never frees or writes caller inputs.
 *   - Streams.  `stream` is a cudaStream_t passed as void*.  Results are ordered
 *     on it: work enqueued on `stream` after a call sees that call's outputs.
 *     fc_score_layer runs power-of-two sequences of 1024..65536 tokens and long
 *     sequences of other lengths on the handle's internal streams (two by
 *     default), which wait for everything enqueued on `stream` before the call
 *     and which `stream` waits for before the call returns, through events; no
 *     host synchronisation is involved (see fc_set_score_overlap for the
 *     variant that defers the second wait).  Nothing uses the default stream.
 *   - Calls that block the host: fc_create and fc_destroy (device
 *     synchronisation), fc_last_device_status and fc_static_last_device_status
 *     (they synchronise `stream`), fc_profile_end (waits for its events),
 *     fc_compress_host (once, to learn the row counts), the first
 *     fc_score_layer_static call on a device.  Every other call only enqueues.
 *   - Context-wide state.  While a handle scores power-of-two sequences it
 *     raises the context's persisting-L2 limit (cudaLimitPersistingL2CacheSize)
 *     to the device maximum and marks its transform workspace as a persisting
 *     access window on its internal streams; the handles of a device share the
 *     claim and the last one to let go restores the value found.  No persisting
 *     line of anyone else is reset.  fc_set_l2_persist(h, 0) opts a handle out.
 *   - Errors.  Argument errors are found on the host before anything is
 *     launched and are returned as fc_status; nothing traps or aborts.  Device-
 *     side problems (capacity overflow, a bounded wait that ran out) set a bit
 *     in the handle's status word, read with fc_last_device_status.  After each
 *     launch the library takes the runtime's pending error (cudaGetLastError):
 *     a non-sticky error left pending by the caller's own earlier CUDA calls is
 *     therefore reported as FC_ERR_CUDA by, and cleared by, the next launch.
 *   - One handle serves one host thread and one stream at a time.
 *   - KV layout: element [t][h][c] at  base + t*stride_token + h*stride_head + c
 *     (strides in elements, channel stride 1).  The sequences of a batch are
 *     packed along t; sequence b owns tokens [cu_seqlens[b], cu_seqlens[b+1]).
 *     Base pointers and row strides must be 16-byte aligned; head_dim must be
 *     a multiple of 64.
 */
#ifndef FLASHCACHE_H_
#define FLASHCACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FC_OK = 0,
  FC_ERR_INVALID_ARG = 1,   /* null pointer, bad size, bad alignment, bad cu_seqlens */
  FC_ERR_UNSUPPORTED = 2,   /* dtype / head_dim / sequence length outside what was built */
  FC_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or smaller than the query says */
  FC_ERR_CUDA = 4,          /* a CUDA runtime call failed */
  FC_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out (set in the status word by the decoding kernel) */
  FC_ERR_INTERNAL = 6       /* a device-side self check failed (see fc_last_device_status) */
} fc_status;

typedef enum { FC_F32 = 0, FC_F16 = 1, FC_BF16 = 2 } fc_dtype;

typedef struct fc_handle fc_handle;   /* opaque: twiddle table, status word, launch counter */
typedef void *fc_stream;              /* a cudaStream_t */

/* One layer's K and V (Eq. 5: K^l = [k_0 .. k_{N-1}], V^l likewise), all KV heads,
 * all sequences of the batch packed along the token axis. */
typedef struct {
  const void *k;              /* DEVICE */
  const void *v;              /* DEVICE */
  int64_t stride_token;       /* elements between consecutive tokens          */
  int64_t stride_head;        /* elements between consecutive heads           */
  int32_t dtype;              /* fc_dtype                                     */
  int32_t num_heads;          /* KV heads H                                   */
  int32_t head_dim;           /* channels per head d                          */
  int32_t batch;              /* number of sequences B                        */
  const int32_t *cu_seqlens;  /* HOST int32[B+1], cu[0] = 0, non-decreasing   */
} fc_kv_view;

/* Create a handle on `device`.  max_seqlen bounds every N_b later passed in
 * (1 <= max_seqlen <= 131072; lengths that are not a power of two, or below 16,
 * are limited to 65536).  Allocates the twiddle table (8 bytes * 4 * next power of two of
 * max_seqlen), room for eight chirp-kernel spectra with their per-row chirp factors (each 8 bytes *
 * (the power of two from 2*max_seqlen-1 up + 2*max_seqlen), at most 2 MiB; lengths that are not a
 * power of two reuse theirs from layer to layer) and a status word.  Returns FC_ERR_CUDA if the device cannot be
 * used, FC_ERR_UNSUPPORTED if max_seqlen is out of range. */
fc_status fc_create(fc_handle **out, int device, int32_t max_seqlen);
void fc_destroy(fc_handle *h);
const char *fc_status_string(fc_status s);

/* Synchronises `stream`, then returns FC_OK or the error the kernels recorded in
 * the handle's device status word since the last call (and clears it). */
fc_status fc_last_device_status(fc_handle *h, fc_stream stream);

/* Measures what the FP32 pipes of this GPU sustain (diagnostic for roofline reports; the paper has no
 * counterpart): a loop of independent fused multiply-adds on every SM, best of three runs of about 2 ms,
 * on the default stream; blocks the host; allocates and frees a small output buffer.  tflops (HOST) counts
 * a fused multiply-add as two operations, like the nominal figure SMs x 128 lanes x 2 x clock. */
fc_status fc_measure_fp32_peak(fc_handle *h, double *tflops);

/* Measurement aid, not on the compression path (the paper has no counterpart): one radix-16 stage of the
 * token-axis transform, y[k][c] = sum_p x[p][c] exp(-2*pi*j*p*k/16), on DEVICE float2 [16][ncols] arrays
 * (ncols a multiple of 8, 16-byte aligned), computed
 *   variant 0  on the FP32 pipes, as the shipped passes do (register-resident butterfly, two columns a thread),
 *   variant 1  on the tensor pipe: the stage as a 32 x 32 real matrix product in TF32 with fp32 accumulation,
 *              operands split in two TF32 terms, three products (about 21 significant bits),
 *   variant 2  not at all (load and store only).
 * repeat > 1 reruns the arithmetic on the loaded registers (timing only; results are then meaningless).
 * Kept so that "FP32 pipes or tensor pipe for a transform stage" stays a measured statement. */
fc_status fc_proto_dft16_stage(fc_handle *h, const void *x, void *y, int32_t ncols, int32_t variant,
                               int32_t repeat, fc_stream stream);

/* Self test of the failure path of the bounded device-side waits (diagnostic; the paper has no
 * counterpart): enqueues one small kernel that waits, at most 1000 tries, on a barrier nothing will ever
 * complete, gives up, and records it.  The next fc_last_device_status returns FC_ERR_TIMEOUT; the
 * context stays usable (nothing traps, nothing spins without a limit). */
fc_status fc_selftest_bounded_wait(fc_handle *h, fc_stream stream);

/* Number of kernels this handle has launched since fc_create (diagnostic). */
uint64_t fc_launch_count(const fc_handle *h);

/* Per-kernel timing (diagnostic; the paper has no counterpart).  Between
 * fc_profile_begin and fc_profile_end every launch of the given kernel class
 * (1 transform pass 1, 2 transform pass 2, 3 transform pass 3 + scoring,
 * 4 top-k selection, 5 row gather, 6 other small kernels) is bracketed by a CUDA
 * event pair on the launching stream, at most max_launches of them.
 * fc_profile_end waits for the recorded events and returns the summed device
 * time in milliseconds and the number of launches timed. */
fc_status fc_profile_begin(fc_handle *h, int32_t kernel_class, int32_t max_launches);
/* Time only every stride-th launch of the class (default 1): the event pairs cost a little and keep
 * neighbouring launches from overlapping, so a sample disturbs a timed region less. */
fc_status fc_profile_stride(fc_handle *h, int32_t stride);
fc_status fc_profile_end(fc_handle *h, double *total_ms, uint64_t *launches);

/* enabled = 1: fc_score_layer calls for power-of-two lengths of 1024..65536 tokens leave their
 * work on the library's two internal streams instead of making `stream` wait for it, so that the
 * next layer starts while the last kernels of this one drain.  Inputs are still taken in stream
 * order (the internal streams wait for everything enqueued on `stream` before the call).  The
 * scores and energies of such calls are ordered on a stream only by the next
 * fc_allocate_budgets, fc_select_compact or fc_last_device_status call that is given that
 * stream; read them earlier only after a device-wide synchronisation.  Default 0: every call
 * is complete in stream order when it returns. */
fc_status fc_set_score_overlap(fc_handle *h, int32_t enabled);

/* enabled = 1: consecutive fc_select_compact calls on one stream may run concurrently (each
 * uses a fraction of the GPU): a launch may begin once every block of the previous one has
 * started, and does not finish before the previous one has, so anything enqueued after the
 * last call still sees all of them complete.  Use it only when (a) nothing else is enqueued on
 * the stream between the calls, and (b) the scores, budgets and offsets of all of them were
 * produced before the first call, as in  score x L, allocate, select x L.  Default 0: every
 * call waits for the one before it. */
fc_status fc_set_select_overlap(fc_handle *h, int32_t enabled);

/* Sequences whose length is not a power of two are transformed by chirp convolutions of a padded
 * power-of-two length (>= 2N - 1).  enabled = 1 (default): where the cutoff index omega of Eq. 8
 * allows a shorter padded length (>= N + 2*omega + 1), only the bins -omega .. omega of the
 * spectrum are computed, the low-pass part (the Base KV of Eq. 9) is transformed back and the
 * score of Eq. 10 is taken against the input rows.  Same result to fp32 rounding; speed only.
 * enabled = 0: always the full-length form (all N bins, residual formed in the frequency domain). */
fc_status fc_set_chirp_band(fc_handle *h, int32_t enabled);

/* Number of internal streams fc_score_layer spreads the head groups of a sequence over (1..4,
 * default 2, the measured best: two transforms in flight fill the GPU, three no longer fit the L2).
 * Call it between passes, not while deferred work is pending (fc_set_score_overlap).  Speed only. */
fc_status fc_set_internal_streams(fc_handle *h, int32_t count);

/* enabled = 0: this handle never touches the context's persisting-L2 limit nor sets access windows
 * (see Conventions); costs a few percent on long power-of-two sequences.  Default 1. */
fc_status fc_set_l2_persist(fc_handle *h, int32_t enabled);

/* Forgets the ordering state the handle keeps between calls (which of its internal events the next
 * call would wait on).  Call it right before cudaStreamBeginCapture and right after
 * cudaStreamEndCapture when a sequence of calls on this handle is captured into a CUDA graph: an
 * event recorded outside a capture cannot be waited on inside one, nor the other way round.
 * Everything enqueued earlier through the handle must already be complete, or be ordered before the
 * next call by the stream that call is given (a graph launch on that stream is). */
fc_status fc_reset_ordering(fc_handle *h);

/* Target size in bytes of the transform intermediates processed per kernel group
 * (kept below the L2 capacity so they are re-read from cache, not HBM).
 * Default 32 MiB.  Affects speed only. */
fc_status fc_set_group_bytes(fc_handle *h, size_t bytes);

/* How a sequence of length seqlen is transformed at cutoff ratio gamma (diagnostic, used for flop
 * accounting; head_dim a multiple of 64 assumed): out = { direct power-of-two path (0), chirp
 * convolutions in the full-length form (1) or in the band form (2, see fc_set_chirp_band),
 * transform length, first factor N1, second factor N2 }. */
fc_status fc_describe_plan(const fc_handle *h, int32_t seqlen, double gamma, int32_t out[4]);

/* Workspace sizes (bytes) the next two calls need for this view.  0 on bad input. */
size_t fc_score_workspace_bytes(const fc_handle *h, const fc_kv_view *kv);
size_t fc_select_workspace_bytes(const fc_handle *h, const fc_kv_view *kv);

/*
 * Outlier KV Recognition Module for one layer (Sec. 3.2.1).
 * For every sequence b (length N), head h and channel c, K and V are taken along
 * the token axis through the orthonormal DCT of Eq. 6-7, low-pass filtered with
 * omega = min(N-1, floor(gamma*N)), bins 0..omega kept (Eq. 8), transformed back
 * (Eq. 9), and every token is scored by
 *     Dev[x] = mean_c (K[x,c]-K_base[x,c])^2 + mean_c (V[x,c]-V_base[x,c])^2   (Eq. 10).
 * Arithmetic is fp32 on the stored values.
 * Values that are not finite: the transform of a channel mixes all tokens of its sequence, so one NaN
 * or Inf element of K or V makes every score of that (sequence, head) NaN and that sequence's energy
 * sums NaN, exactly as the definition does; other heads' scores and other sequences are unaffected.
 * fc_allocate_budgets then treats the sequence's weights as uniform and fc_select_compact ranks NaN as
 * +inf, ties by token index: the affected head keeps its first tokens.
 *
 *   gamma      cutoff factor, 0 <= gamma <= 1.
 *   scores     DEVICE float[num_heads][T], T = cu_seqlens[B]; written for every token.
 *   energy     DEVICE double[B][4] = (hiK, totK, hiV, totV) per sequence: the sums of the
 *              power spectrum P[m] = |C[m]|^2 (Eq. 11) over m > omega and over all m, over
 *              every head and channel of the layer -- numerators and denominators of
 *              Eq. 12.  By Parseval (the orthonormal transform of Eq. 6-7) they are
 *              accumulated as d*sum Dev_k and sum K^2 without storing a spectrum.
 *   workspace  DEVICE, 256-byte aligned, >= fc_score_workspace_bytes(); scratch only.
 * Errors: FC_ERR_INVALID_ARG, FC_ERR_UNSUPPORTED (dtype, head_dim % 64, N_b > max_seqlen),
 * FC_ERR_WORKSPACE, FC_ERR_CUDA (launch failure).
 */
fc_status fc_score_layer(fc_handle *h, const fc_kv_view *kv, double gamma,
                         float *scores, double *energy,
                         void *workspace, size_t workspace_bytes, fc_stream stream);

/*
 * Dynamic Budget Allocation Module (Sec. 3.2.2): R^l = hiK/totK + hiV/totV (Eq. 12)
 * per layer and sequence, normalised to weights, the total budget
 * B_tot = clamp(floor(rho*N*L + 1/2), L*lo, L*N), lo = min(min_keep, N), shared out as
 * q_l = clamp(lambda*w_l, lo, N) with sum q_l = B_tot, made integer by largest
 * remainder (ties: lower layer first).  All in fp64 on the device.
 *
 *   energy           DEVICE double[L][B][4] (the per-layer outputs of fc_score_layer).
 *   cu_seqlens_host  HOST int32[B+1].
 *   budgets          DEVICE int32[L][B]: tokens kept per head in layer l, sequence b.
 *   out_offsets      DEVICE int64[L][B+1]: exclusive prefix sum of budgets[l][.]
 *                    (first row of sequence b in layer l's compacted cache; [B] = rows).
 * Limits: 1 <= L <= 1024.  Errors: FC_ERR_INVALID_ARG, FC_ERR_UNSUPPORTED, FC_ERR_CUDA.
 */
fc_status fc_allocate_budgets(fc_handle *h, const double *energy, int32_t num_layers,
                              int32_t batch, const int32_t *cu_seqlens_host,
                              double rho, int32_t min_keep,
                              int32_t *budgets, int64_t *out_offsets, fc_stream stream);

/*
 * Keep the Outlier KVs of one layer (Sec. 3.2.1, last sentence; compacted cache of
 * Fig. 2): for every sequence b and head h the budgets[b] tokens with the largest
 * score (order: score descending, token index ascending; NaN ranks as +inf) are
 * written as ascending sequence-local token indices, and their K and V rows are
 * copied bit for bit.
 *
 *   scores       DEVICE float[num_heads][T]           (from fc_score_layer)
 *   budgets      DEVICE int32[B]                      (layer l's slice)
 *   out_offsets  DEVICE int64[B+1]                    (layer l's slice)
 *   out_idx      DEVICE int32[num_heads][out_capacity_rows]; entry [h][out_offsets[b]+j]
 *   out_k,out_v  DEVICE, dtype of the input, dense [row][h][c], out_capacity_rows rows;
 *                row out_offsets[b]+j, head h = input row cu[b]+out_idx[h][..], head h.
 *   out_capacity_rows  rows available; a sequence whose rows would pass it is
 *                skipped and FC_ERR_INTERNAL is recorded in the status word.
 *   workspace    DEVICE, 256-byte aligned, >= fc_select_workspace_bytes().
 */
fc_status fc_select_compact(fc_handle *h, const fc_kv_view *kv, const float *scores,
                            const int32_t *budgets, const int64_t *out_offsets,
                            void *out_k, void *out_v, int32_t *out_idx,
                            int64_t out_capacity_rows,
                            void *workspace, size_t workspace_bytes, fc_stream stream);

/*
 * Spectrum diagnostics (Sec. 3.2.2, Eq. 11; the curves of the paper's energy-distribution figures):
 * the power spectrum of one layer, P_k[m] = |C_k[m]|^2 and P_v[m] = |C_v[m]|^2, where C[m] is the row of
 * DCT coefficients (Eq. 6-7) of frequency m over all channels of all KV heads.  Its band sums are the
 * numerators and denominators of Eq. 12 (what fc_score_layer returns as `energy`), its running sum is
 * the cumulative-energy curve from which a cutoff gamma can be read.  Not on the compression path:
 * it runs the generic transform kernels on the caller's stream.
 *
 *   spectrum   DEVICE double[T][2]: row cu_seqlens[b] + m = (P_k[m], P_v[m]) of sequence b.
 *   workspace  DEVICE, 256-byte aligned, >= fc_power_spectrum_workspace_bytes().
 * Errors: as fc_score_layer.
 */
size_t fc_power_spectrum_workspace_bytes(const fc_handle *h, const fc_kv_view *kv);
fc_status fc_power_spectrum(fc_handle *h, const fc_kv_view *kv, double *spectrum,
                            void *workspace, size_t workspace_bytes, fc_stream stream);

/*
 * Cutoff read from the spectrum (Sec. 3.2.2, Eq. 11-12; the energy-distribution figures; the gamma
 * ablation of Sec. 4.3): for every sequence the smallest omega whose kept band 0..omega (Eq. 8) holds at
 * least `share` of the total energy sum_m P_k[m] + P_v[m], i.e. the smallest cutoff that leaves at most
 * 1 - share of the energy to the outlier band of Eq. 12.
 *
 *   spectrum    DEVICE double[T][2] as written by fc_power_spectrum
 *   cu_seqlens  HOST int32[batch+1]
 *   share       0 <= share <= 1
 *   omega       DEVICE int32[batch]
 *   gamma       DEVICE double[batch] = (omega + 1/2) / N: passed to fc_score_layer it gives exactly this
 *               omega (min(N-1, floor(gamma*N))); an empty sequence gets 0, a spectrum without energy omega 0
 * fp64 running sums in a fixed order.  Errors: FC_ERR_INVALID_ARG, FC_ERR_CUDA.
 */
fc_status fc_cutoff_from_spectrum(fc_handle *h, const double *spectrum, int32_t batch,
                                  const int32_t *cu_seqlens, double share, int32_t *omega,
                                  double *gamma, fc_stream stream);

/*
 * Decoding step on the compacted cache (Sec. 3.1, Eq. 3-4): for every sequence b and query head j
 *     out[b][j] = Softmax(q[b][j] K^T / sqrt(head_dim)) V
 * where K and V are, for KV head j / (num_q_heads / num_heads), the rows the compressor kept for
 * sequence b (rows offsets[b] .. offsets[b+1] of one layer's compacted cache, as written by
 * fc_select_compact) followed by the KV pairs appended since the prefill, which stay uncompressed
 * (the `tail`).  Reads every K and V row once; fp32 accumulation; a sequence without rows gives zeros.
 *
 *   q            DEVICE [batch][num_q_heads][head_dim], dtype FC_F16 or FC_BF16 (as the cache)
 *   cache_k/v    DEVICE [cache_rows][num_heads][head_dim] dense, 16-byte aligned
 *   offsets      DEVICE int64[batch+1] (one layer's slice of fc_allocate_budgets' out_offsets)
 *   tail_k/v     DEVICE [batch][tail_capacity][num_heads][head_dim] or NULL
 *   tail_len     DEVICE int32[batch]: valid rows of each sequence's tail (<= tail_capacity)
 *   max_rows     HOST upper bound of (kept rows + tail rows) of any sequence; sizes the launch only
 *   out          DEVICE [batch][num_q_heads][head_dim], same dtype
 *   workspace    DEVICE, 256-byte aligned, >= fc_decode_workspace_bytes()
 * Limits: head_dim 128, num_q_heads a multiple of num_heads with at most 16 query heads per KV head.
 * Errors: FC_ERR_INVALID_ARG, FC_ERR_UNSUPPORTED, FC_ERR_WORKSPACE, FC_ERR_CUDA; a bounded wait that
 * runs out sets FC_ERR_TIMEOUT in the device status word.
 */
typedef struct {
  const void *q;
  const void *cache_k, *cache_v;
  int64_t cache_rows;
  const int64_t *offsets;
  const void *tail_k, *tail_v;
  const int32_t *tail_len;
  int32_t tail_capacity;
  int32_t dtype, batch, num_heads, num_q_heads, head_dim;
  int64_t max_rows;
} fc_decode_args;

size_t fc_decode_workspace_bytes(const fc_handle *h, const fc_decode_args *a);
fc_status fc_decode_attention(fc_handle *h, const fc_decode_args *a, void *out,
                              void *workspace, size_t workspace_bytes, fc_stream stream);

/*
 * fc_select_compact with options (opt == NULL: exactly fc_select_compact).
 *
 *   per_layer  0: every KV head keeps its own tokens (the default reading: Eq. 10 over the head's
 *              d channels).  1: the layer-wide reading of Sec. 3.1 / Eq. 5, where K^l is N x D with
 *              D the whole hidden width: one index set per layer and sequence, ranked by the
 *              deviation over all H*d channels, i.e. by the mean (here: the sum, same order) over
 *              the heads of the per-head scores; every head keeps those tokens, out_idx holds the
 *              same indices for every head.
 *   protect    DEVICE uint8[T] or NULL.  A non-zero byte marks a token that must survive (text
 *              tokens, attention sinks, a recent window; the paper compresses the visual KVs,
 *              Sec. 1): it ranks before every unmarked token, marked tokens rank among themselves
 *              by index.  The budget still counts them: a sequence with more marked tokens than
 *              budget keeps the first `budget` of them, so give fc_allocate_budgets a min_keep of
 *              at least the largest number of marked tokens in a sequence.
 */
typedef struct {
  int32_t per_layer;
  const void *protect;
} fc_select_options;

fc_status fc_select_compact_ex(fc_handle *h, const fc_kv_view *kv, const float *scores,
                               const int32_t *budgets, const int64_t *out_offsets,
                               void *out_k, void *out_v, int32_t *out_idx,
                               int64_t out_capacity_rows, const fc_select_options *opt,
                               void *workspace, size_t workspace_bytes, fc_stream stream);

/*
 * fc_select_compact_ex for several layers in ONE launch (Sec. 3.2.1, last sentence; same selection, same
 * results bit for bit).  After fc_allocate_budgets every layer's scores, budgets and offsets are known, and
 * one layer's selection fills only a fraction of the GPU (8 blocks per sequence and head), so the layers
 * are best selected side by side.
 *
 *   shape        the layout all layers share: strides, dtype, num_heads, head_dim, batch, cu_seqlens
 *                (its k and v are not read)
 *   layers       HOST array [num_layers] of per-layer DEVICE pointers and the rows available in that
 *                layer's outputs (copied into the launch arguments; free to reuse on return)
 *   budgets      DEVICE int32[num_layers][B], out_offsets DEVICE int64[num_layers][B+1]: the arrays
 *                fc_allocate_budgets wrote (row l belongs to layers[l])
 *   opt          as fc_select_compact_ex (NULL: defaults); the protect mask is shared by all layers
 * Layers are launched 32 at a time.  Errors: as fc_select_compact_ex.
 */
typedef struct {
  const void *k, *v;           /* DEVICE: the layer's K and V                      */
  const float *scores;         /* DEVICE float[num_heads][T] from fc_score_layer   */
  void *out_k, *out_v;         /* DEVICE [out_capacity_rows][h][c]                 */
  int32_t *out_idx;            /* DEVICE int32[num_heads][out_capacity_rows]       */
  int64_t out_capacity_rows;
} fc_layer_buffers;

fc_status fc_select_compact_layers(fc_handle *h, const fc_kv_view *shape, const fc_layer_buffers *layers,
                                   int32_t num_layers, const int32_t *budgets, const int64_t *out_offsets,
                                   const fc_select_options *opt, void *workspace, size_t workspace_bytes,
                                   fc_stream stream);

/* Rows one layer's compacted cache can receive at most: the sum over sequences of
 * min(N_b, B_tot(b)), B_tot = clamp(floor(rho*N*L + 1/2), L*lo, L*N) (Sec. 3.2.2; the total the
 * budgets of a sequence add up to).  Sizes out_k / out_v / out_idx before the budgets are known.
 * -1 on bad input. */
int64_t fc_layer_capacity_rows(int32_t num_layers, int32_t batch, const int32_t *cu_seqlens,
                               double rho, int32_t min_keep);

/*
 * fc_score_layer without any allocation (the paper has no counterpart: this is a
 * packaging variant of the same computation, added for integration reasons).
 *
 * Who needs it: code that is not allowed to obtain device memory at the point where it
 * wants to score a layer -- for example a serving process whose whole device memory is
 * handed to a framework's pool at start-up, a plug-in interface that forbids allocation
 * after initialisation, or a real-time path where the implicit device synchronisation
 * of cudaMalloc/cudaFree is not acceptable.  Such callers cannot use fc_create (it
 * allocates the twiddle table) nor provide the workspace of fc_score_layer.
 *
 * This entry point needs no handle and no workspace.  Its twiddle table and all of its
 * scratch live in arrays that are part of the library image: FC_STATIC_SCRATCH_BYTES
 * (8 MiB) of scratch plus a 128 KiB table, held by every GPU that has loaded the library
 * until the process exits.  It calls no cudaMalloc, cudaFree or other allocating routine.
 * Inputs and outputs are the caller's, exactly as for fc_score_layer:
 *
 *   kv, gamma, scores, energy, stream   as in fc_score_layer (same layout, same results
 *                                       up to fp32 rounding: it runs the library's generic
 *                                       transform kernels for every length).
 *
 * Limits: every sequence length <= 4096 (else FC_ERR_UNSUPPORTED), and the scratch the view
 * needs (what fc_score_workspace_bytes would report with one head per transform group)
 * <= FC_STATIC_SCRATCH_BYTES (else FC_ERR_WORKSPACE).  A power-of-two length N needs
 * N * head_dim * 8 bytes plus a few KiB (at head_dim 128: up to 4096; at 256: up to 2048);
 * any other length up to 4096 fits at every head_dim (a head is transformed 32 columns at a
 * time).
 *
 * First call on a device: looks up the device addresses of the arrays, fills the twiddle
 * table and waits for the device once (cudaDeviceSynchronize).  Make that first call with
 * the device current and before any stream capture begins.  Later calls only enqueue
 * kernels on `stream`.
 *
 * Sharing: all calls on one device use the same scratch, which keeps the previous call's
 * contents (every region is rewritten before it is read, nothing needs clearing).  Two
 * calls that can overlap on the GPU (different streams, or different host threads without
 * ordering between their streams) race on it; order them.
 */
#define FC_STATIC_SCRATCH_BYTES ((size_t)8 << 20)
size_t fc_static_scratch_bytes(void);
fc_status fc_score_layer_static(const fc_kv_view *kv, double gamma, float *scores,
                                double *energy, fc_stream stream);
/* fc_last_device_status for the calls above (they have no handle): synchronises `stream`, returns and
 * clears what the kernels of fc_score_layer_static recorded in the status word of the current device. */
fc_status fc_static_last_device_status(fc_stream stream);

/*
 * The whole compressor for one prefill, from HOST memory to HOST memory (Sec. 3.2, Fig. 2):
 * copies every layer's K and V to the device, scores each layer as soon as its copies have
 * landed (fc_score_layer), allocates the budgets over all layers (fc_allocate_budgets), keeps
 * the Outlier KVs of every layer (fc_select_compact) and copies the compacted caches back.
 * The same kernels as the per-stage entry points, so the same results; what this call adds is
 * the copy pipeline around them.
 *
 * Inputs (HOST; page-locked memory lets the copies overlap the kernels, pageable memory
 * works but serialises them):
 *   k_host, v_host   [num_layers] pointers; layer l dense [T][num_heads][head_dim] of `dtype`,
 *                    T = cu_seqlens[batch].
 *   cu_seqlens       int32[batch+1], as in fc_kv_view.
 *   gamma, rho, min_keep   as in fc_score_layer and fc_allocate_budgets.
 *   per_layer, protect_host   the options of fc_select_compact_ex; protect_host is a HOST uint8[T]
 *                    mask (or NULL) that the call copies to the device with the inputs.
 * Device memory (DEVICE, owned by the caller, 256-byte aligned, >= fc_compress_host_arena_bytes):
 *   arena            staging for the inputs of all layers, scores, energies, budgets, the
 *                    compacted caches and the kernels' workspace.  Two consecutive calls with
 *                    the same arena are ordered by the library (the second call's copies wait
 *                    for the first call's selection, not for its copies back to the host, so
 *                    they overlap those).  Otherwise the arena must not be in use by work that
 *                    was enqueued later than the moment `stream` has reached at the call.
 * Outputs (HOST, valid once `stream` has been synchronised after the call):
 *   budgets_host     int32[num_layers][batch]     tokens kept per head (layer, sequence)
 *   offsets_host     int64[num_layers][batch+1]   prefix sums, as fc_allocate_budgets' out_offsets
 *   layer_rows_host  int64[num_layers+1]          first packed row of every layer; [L] = rows in all
 *   out_k_host, out_v_host   packed rows [row][num_heads][head_dim]; layer l, sequence b, j-th
 *                    kept token = row layer_rows[l] + offsets[l][b] + j
 *   out_idx_host     int32; layer l's indices are the array [num_heads][r_l], r_l =
 *                    layer_rows[l+1]-layer_rows[l], starting at element num_heads*layer_rows[l];
 *                    entry [h][offsets[l][b]+j] = sequence-local token index, ascending in j
 *   out_capacity_rows  rows available in out_k_host / out_v_host (and num_heads times as many
 *                    index entries); fc_compress_host_rows() gives the number needed.
 * budgets_host, offsets_host and layer_rows_host are already valid when the call returns: the call
 * blocks the host once, after the budgets are known, to learn the sizes of the copies back.
 * (For that reason the call cannot be captured into a CUDA graph; the per-stage entry points can.)
 *
 * Errors: FC_ERR_INVALID_ARG, FC_ERR_UNSUPPORTED (as fc_score_layer), FC_ERR_WORKSPACE (arena
 * too small or misaligned; more rows than out_capacity_rows, in which case nothing is copied
 * back), FC_ERR_CUDA.  Device-side checks report through fc_last_device_status as usual.
 */
typedef struct {
  const void *const *k_host;
  const void *const *v_host;
  int32_t num_layers, dtype, num_heads, head_dim, batch, min_keep;
  const int32_t *cu_seqlens;
  double gamma, rho;
  void *arena;
  size_t arena_bytes;
  void *out_k_host, *out_v_host;
  int32_t *out_idx_host;
  int64_t out_capacity_rows;
  int32_t *budgets_host;
  int64_t *offsets_host;
  int64_t *layer_rows_host;
  int32_t per_layer;
  const uint8_t *protect_host;
} fc_host_job;

/* Rows the compacted caches of all layers hold together: the sum over sequences of
 * B_tot = clamp(floor(rho*N*L + 1/2), L*lo, L*N) (Sec. 3.2.2), which the budgets add up to. */
int64_t fc_compress_host_rows(int32_t num_layers, int32_t batch, const int32_t *cu_seqlens,
                              double rho, int32_t min_keep);
/* Device bytes fc_compress_host needs for this job (only the shape fields, cu_seqlens, rho and
 * min_keep are read).  0 on bad input. */
size_t fc_compress_host_arena_bytes(const fc_handle *h, const fc_host_job *job);
fc_status fc_compress_host(fc_handle *h, const fc_host_job *job, fc_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* FLASHCACHE_H_ */
