/*
 * prox.h - C ABI of libprox: the decode-time sparse SwiGLU FFN of "Prox"
 * (training-free FFN activation sparsity through an approximate
 * intermediate-channel salience), written for one NVIDIA B200 (sm_100a).
 *
 * The path (paper Sec. 4.1 "Two-Stage Sparse Inference"):
 *   Stage 1  proxy mask:  m_x keeps the k1 largest |x_i|; the quantized proxy
 *            copies of W_gate and W_up are multiplied against the kept inputs
 *            only (input sparsity Pi_in, Sec. 2.2); the proxy state
 *            s~ = u~ (.) SiLU(g~) is ranked by magnitude and the k2 largest
 *            channels form the mask m_s shared by all three projections.
 *   Stage 2  exact sparse compute:  for the channels in m_s, gate and up are
 *            recomputed with the original bf16 weights and the dense x
 *            (output sparsity Pi_out), s = u (.) SiLU(g), and the down
 *            projection sums s_j * W_down[j,:] over those channels only.
 *
 * Selection rule: the paper's main rule is a calibrated layer threshold
 * (indicator |z| >= tau); this library implements the per-token top-k rule of
 * the appendix "Threshold-Based Selection and Token-Adaptive Computation"
 * (exactly k entries, ties go to the lower index) and, as a variant, the
 * threshold rule with caller-supplied tau (prox_*_threshold entry points).
 *
 * Conventions for every call
 *   - "dev" pointers are CUDA device pointers on the current device, "host"
 *     pointers are ordinary host memory.  Nothing here takes a framework type.
 *   - Matrices are row-major with the nn.Linear orientation:
 *       W_gate, W_up : bf16 [d_ff, d_model]   row j = weights of channel j
 *       W_down       : bf16 [d_model, d_ff]
 *     (the paper writes W_up, W_gate in R^{d_model x d_ff}, W_down in
 *     R^{d_ff x d_model}; these are the transposes, Sec. 2.1).
 *   - x is bf16 [B, d_model]; y is [B, d_model] in the handle's out_dtype.
 *     Each of the B tokens gets its own masks (the paper covers B = 1 only).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work
 *     is enqueued on it and the call returns without synchronising unless the
 *     call's comment says otherwise.  A handle must not be used from two
 *     streams at once: its scratch buffers are shared by all calls.
 *   - Every call validates its arguments on the host and returns a status;
 *     nothing throws or aborts across this boundary.  Inputs are assumed
 *     finite; NaN/Inf in x or the weights give unspecified masks.
 *   - Caller-owned memory: x, y, sel, scores and the original weights.
 *     w_gate and w_up are BORROWED for the handle's whole life (Stage 2 reads
 *     them in place); w_down is read only by prox_quantize_proxy.  The handle
 *     owns the packed proxies, their scales, the channel-major copy of W_down
 *     and all scratch.
 */
#ifndef PROX_H_
#define PROX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct prox_ffn prox_ffn_t;

typedef enum {
  PROX_OK = 0,
  PROX_ERR_INVALID_ARG = 1,   /* null pointer, size out of range, misaligned pointer */
  PROX_ERR_UNSUPPORTED = 2,   /* shape / bits / group_size this build does not handle */
  PROX_ERR_NOT_QUANTIZED = 3, /* Stage 1 asked for before prox_quantize_proxy */
  PROX_ERR_CUDA = 4,          /* a CUDA runtime call failed (incl. no device) */
  PROX_ERR_OOM = 5,           /* device or host allocation failed */
  PROX_ERR_TIMEOUT = 6,       /* a bounded device-side wait gave up */
  PROX_ERR_IO = 7             /* file could not be read / written / parsed */
} prox_status_t;

typedef struct {
  int32_t d_model;   /* D: multiple of 128, 128..16384 */
  int32_t d_ff;      /* F: multiple of 64,  64..65536  */
  int32_t max_batch; /* 1..8 tokens per call */
  int32_t out_dtype; /* 0 = bf16, 1 = fp32 */
} prox_ffn_config_t;

/* Create a handle over caller-owned dev bf16 weights (Sec. 2.1 for the shapes).
 * Pointers must be 16-byte aligned.  Allocates scratch; copies nothing.
 * Errors: INVALID_ARG, UNSUPPORTED (shape), CUDA, OOM. */
prox_status_t prox_ffn_create(const prox_ffn_config_t* cfg, const void* w_gate_dev,
                              const void* w_up_dev, const void* w_down_dev,
                              void* stream, prox_ffn_t** out);

/* Offline packer (Sec. 4.3: "symmetric per-row INT4 quantization of the
 * original W_up and W_gate ... keeping the compact proxies resident in GPU
 * memory").  For every channel j and every group of `group_size` consecutive
 * input indices (0 = the whole row, the paper's per-row case):
 *     scale = fp16(max|w| / qmax),  qmax = 2^(bits-1)-1
 *     q     = clamp(rint(w / scale), -qmax, qmax)      (fp32, ties to even)
 * Proxies are stored input-major (all channels of one input coordinate are
 * contiguous, gate and up interleaved) so that Stage 1's input sparsity skips
 * whole rows of bytes.  Also writes the channel-major copy of W_down
 * ([d_ff, d_model], Sec. 3.1: y = sum_j s_j W_down[j,:]) so that the masked
 * down projection reads one contiguous row per kept channel.
 * bits in {4, 8}; group_size in {0, 128}.  May be called again to re-pack.
 * bits = 16 (group_size 0 only) stores the original bf16 weights themselves in
 * the same input-major order, with no scales: the 16-bit proxy of ablation A1
 * (Sec. "Ablation Studies"), and the 16-bit input-sparse GEMV that the cost
 * ratio alpha of Sec. 4.2 compares the integer proxy GEMV with.  With 16-bit
 * proxies the forward calls take the step-wise kernels (the fused kernel and
 * the batched Stage 1 read integer codes); prox_proxy_export is UNSUPPORTED.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA, OOM. */
prox_status_t prox_quantize_proxy(prox_ffn_t* h, int bits, int group_size, void* stream);

/* Stage 1 (Sec. 4.1, "lightweight proxy construction"), top-k rule.
 *   x          dev bf16 [B, D]
 *   k1         kept inputs per token, 1..D   (k1 = D keeps every input)
 *   k2         kept channels per token, 1..F
 *   sel        dev int32 [B, k2] out: kept channel ids, ascending, per token
 *   scores     dev fp32 [B, F] out or NULL: |u~_j * SiLU(g~_j)|
 * Errors: INVALID_ARG, NOT_QUANTIZED, CUDA. */
prox_status_t prox_stage1_mask(prox_ffn_t* h, const void* x_dev, int B, int k1, int k2,
                               int32_t* sel_dev, float* scores_dev_or_null, void* stream);

/* Stage 2 (Sec. 4.1, "exact sparse computation") for a given mask.
 *   sel        dev int32 [B, k2]: channel ids per token, each in [0, F),
 *              ascending and unique within a token (as Stage 1 writes them)
 *   y          dev [B, D] out, out_dtype
 * Out-of-range ids are skipped and recorded (see prox_last_device_status).
 * Needs the channel-major W_down, i.e. prox_quantize_proxy must have run.
 * Errors: INVALID_ARG, NOT_QUANTIZED, CUDA. */
prox_status_t prox_stage2_ffn(prox_ffn_t* h, const void* x_dev, int B, const int32_t* sel_dev,
                              int k2, void* y_dev, void* stream);

/* Stage 1 then Stage 2 on one stream; the mask stays on the device. */
prox_status_t prox_ffn_forward(prox_ffn_t* h, const void* x_dev, int B, int k1, int k2,
                               void* y_dev, void* stream);

/* For B = 1 prox_ffn_forward runs the whole path as ONE persistent kernel
 * (cooperative launch, one block per SM, one grid-wide barrier with a bounded
 * wait between Stage 1 and Stage 2); prox_ffn_set_fused(h, 0) selects the
 * kernel-per-step path instead (always used for B > 1).  If a bounded wait
 * ever expires the kernel leaves, y is not written (undefined) and
 * prox_last_device_status reports bit 4 and returns PROX_ERR_TIMEOUT. */
prox_status_t prox_ffn_set_fused(prox_ffn_t* h, int on);

/* Mask policy of calls with B > 1 (the paper treats batch 1 only and names batching as future work):
 *   0  every token its own channel mask (default; a token's result is the one it would get alone)
 *   1  one channel mask for the batch: the k2 channels of largest summed proxy score
 *      sum_b |s~_{b,j}| (ties: lower channel); input masks and proxy scores stay per token, and
 *      Stage 2 reads k2 rows instead of the union of B masks.  Built by the tensor-core batch
 *      path (4-bit proxies); other configurations return UNSUPPORTED from the forward calls.
 * B = 1 is not affected.  Errors: INVALID_ARG. */
prox_status_t prox_ffn_set_mask_policy(prox_ffn_t* h, int policy);

/* For B > 1 every token keeps its own masks (the paper covers B = 1 only), and the
 * weights are read once per call for the UNION of the tokens' kept inputs and of
 * their kept channels; a token contributes zero outside its own masks, so its
 * result is the one it would get alone.  With the union, the exact Stage 2
 * runs as warp-level bf16 tensor-core tiles (16 channels x 8 tokens x 16 inputs)
 * with fp32 accumulation; in the down projection h enters as a bf16 pair
 * hi + lo.  prox_ffn_set_union(h, 1) keeps the union but computes with plain fp32
 * FMAs, prox_ffn_set_union(h, 0) selects the older path that runs the
 * single-token kernels once per token; any other value (the default) selects the
 * tensor-core union path. */
prox_status_t prox_ffn_set_union(prox_ffn_t* h, int on);

/* Launch plan of the persistent kernel for budgets (k1, k2), for diagnostics:
 * info[8] (host) = {usable, grid blocks, row split, dynamic shared bytes, ring
 * slots, registers per thread, static shared bytes, co-resident blocks per SM}. */
prox_status_t prox_fused_kernel_info(prox_ffn_t* h, int k1, int k2, int32_t* info_host);

/* Debug aid: with on != 0 every block of the persistent kernel records time
 * stamps (nanoseconds of the GPU's global timer) per call.  Slots 0..9: kernel
 * entry, end of set-up, of the input mask, of the proxy GEMV, of the grid
 * barrier, of the channel mask (as seen by thread 0, which helps to settle the
 * threshold bin), slot 6 end of that settling, 7 last row consumed, 8 partial-y
 * exchange done, 9 finalize done (last block only).  Slots 10..31 are finer
 * marks inside those phases (16..21: front part of the channel mask, 21 = go
 * flag for the ring; 28 / 30: first copy / first down-projection row armed by a
 * producer warp).  If stamps_host is given, the stamps of the last call are
 * copied to it as [min(max_blocks, SM count)][32] uint64 (synchronises).
 * on = 0 frees the buffer. */
prox_status_t prox_fused_trace(prox_ffn_t* h, int on, uint64_t* stamps_host, int max_blocks);

/* Test hook: what Stage 1 of the most recent forward call at B = 1 itself computed: its kept-input
 * list (first indicator of Sec. 4.1; dev int32 [k1], ascending; NULL to skip) and its proxy scores
 * (|u~ SiLU(g~)|, dev fp32 [d_ff]; NULL to skip).  Enqueued on stream. */
prox_status_t prox_ffn_last_stage1(prox_ffn_t* h, int k1, int32_t* idx_dev_or_null, float* scores_dev_or_null,
                                   void* stream);

/* Test hook for the bounded device-side waits: spin_limit = polls after which a wait gives up
 * (0 = the default, about two million); barrier_bias > 0 keeps the grid barrier of the persistent
 * kernel from ever completing, so that the next B = 1 forward call runs into the limit, leaves
 * without writing y and reports it (see prox_last_device_status).  Nothing hangs or faults: the
 * blocks give up and return.  Set both back to 0 afterwards. */
prox_status_t prox_debug_set_wait(prox_ffn_t* h, uint32_t spin_limit, uint32_t barrier_bias);

/* Copy the channel mask of the most recent prox_ffn_forward call (top-k rule)
 * into sel_dev, dev int32 [B, k2], ascending per token.  Enqueued on stream. */
prox_status_t prox_ffn_last_mask(prox_ffn_t* h, int B, int k2, int32_t* sel_dev, void* stream);

/* Same as prox_ffn_forward with HOST buffers: copies x (host bf16 [B, D]) to
 * the device, runs the path, brings y back and synchronises the stream before
 * returning.  Pinned host memory makes the copies asynchronous w.r.t. other
 * streams, and a pinned (mapped) y_host is written by the kernels directly, with
 * no copy back; pageable memory also works. */
prox_status_t prox_ffn_forward_host(prox_ffn_t* h, const void* x_host, int B, int k1, int k2,
                                    void* y_host, void* stream);

/* Stage 2 for callers that must not allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of prox_stage2_ffn.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a
 * framework's stream-ordered or graph-captured region, under a memory pool that
 * owns the whole device, in a latency-critical serving loop that forbids
 * allocator calls, or in a plug-in that is handed raw buffers and no handle.
 * Such a caller cannot create a prox_ffn_t (creating one allocates).
 *
 * What it does: for one token (B = 1) it computes h_j = SiLU(x . W_gate[j,:]) *
 * (x . W_up[j,:]) for the k2 channels in sel and y = sum_j h_j W_down_t[j,:],
 * exactly like prox_stage2_ffn, but takes every tensor from the caller:
 *   x            dev bf16 [d_model]
 *   w_gate, w_up dev bf16 [d_ff, d_model]
 *   w_down_t     dev bf16 [d_ff, d_model]: W_down stored channel-major (row j is
 *                the d_model weights of channel j, i.e. the transpose of the
 *                [d_model, d_ff] matrix the other entry points take)
 *   sel          dev int32 [k2], ids in [0, d_ff) (others are skipped)
 *   y            dev [d_model], bf16 (out_dtype 0) or fp32 (1)
 * The two intermediates (one fp32 h per kept channel and the fp32 accumulator of
 * y) live in a 192 KB array that is part of the library image on every GPU that
 * loads it, instead of in allocated memory.  Hence the limits: d_model <= 16384
 * and k2 <= 32768 (PROX_ERR_UNSUPPORTED beyond; use the handle-based call).
 * No cudaMalloc, cudaFree or allocating library routine is called.
 *
 * The first call on a device looks up the device address of that array (the
 * device must be current); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the last call's
 * contents (the accumulator is cleared at the start of every call): two calls
 * that overlap on the GPU - different streams, or concurrent host threads -
 * race on it, so serialise them.  Work is enqueued on `stream`; no sync.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
prox_status_t prox_stage2_ffn_noalloc(const void* x_dev, const void* w_gate_dev, const void* w_up_dev,
                                      const void* w_down_t_dev, int d_model, int d_ff,
                                      const int32_t* sel_dev, int k2, void* y_dev, int out_dtype,
                                      void* stream);

/* Threshold variant of the two indicators of Sec. 4.1:
 *   [m_x]_i = 1[|x_i| >= tau_x],  [m_s]_j = 1[|s~_j| >= tau_s].
 * The number of kept entries varies per token.
 *   count_dev  dev int32 [B] out: kept channels per token
 *   sel        dev int32 [B, F] out: first count[b] entries of row b are valid
 * prox_stage2_ffn_var consumes that layout (row stride F). */
prox_status_t prox_stage1_mask_threshold(prox_ffn_t* h, const void* x_dev, int B, float tau_x,
                                         float tau_s, int32_t* sel_dev, int32_t* count_dev,
                                         float* scores_dev_or_null, void* stream);
prox_status_t prox_stage2_ffn_var(prox_ffn_t* h, const void* x_dev, int B, const int32_t* sel_dev,
                                  const int32_t* count_dev, void* y_dev, void* stream);
/* prox_ffn_forward_threshold at B = 1 is one launch of the persistent kernel in
 * its threshold form (no k-th element search); the mask it used can be read with
 * prox_ffn_last_mask(h, 1, n, ...) where n is the kept-channel count that
 * prox_runtime_sparsity reports, and is ascending.  Otherwise it is
 * prox_stage1_mask_threshold followed by prox_stage2_ffn_var. */
prox_status_t prox_ffn_forward_threshold(prox_ffn_t* h, const void* x_dev, int B, float tau_x,
                                         float tau_s, void* y_dev, void* stream);

/* Ablation A3 of Sec. "Ablation Studies" (necessity of exact computation):
 * Stage 1 as in prox_ffn_forward, then the signed proxy values
 * s~_j = u~_j SiLU(g~_j) of the k2 selected channels enter the down projection,
 *     y = sum_{j in m_s} s~_j W_down[j,:],
 * and the exact gate/up of Stage 2 is skipped.  With 16-bit proxies this is the
 * pattern Sec. 2.2 attributes to TEAL: input sparsity on x for gate/up, then
 * input sparsity on the resulting s for the down projection.
 * Arguments, layouts and errors as prox_ffn_forward; step-wise kernels. */
prox_status_t prox_ffn_forward_proxy_values(prox_ffn_t* h, const void* x_dev, int B, int k1, int k2,
                                            void* y_dev, void* stream);

/* One layer's FFN sub-block on the residual stream (pre-norm decoder layer; the
 * appendix "End-to-End Latency Analysis" counts RMSNorm and the residual around
 * the FFN into the per-token time of a layer):
 *     x_res' = x_res + ProxFFN( bf16( x_res / sqrt(mean(x_res^2) + eps) * norm_w ) ).
 *   x_res      dev fp32 [B, d_model]  the residual stream (read)
 *   norm_w     dev bf16 [d_model]     RMSNorm weight
 *   x_res_out  dev fp32 [B, d_model]  result; may be x_res itself (in place)
 * The norm is evaluated in fp64 and rounded once to bf16, so that the FFN input,
 * on which both masks depend, is the nearest bf16 of the exact value.  At B = 1
 * norm, FFN and residual add are one launch of the persistent kernel; otherwise
 * one small norm kernel precedes the batch path and its last kernel adds x_res.
 * The handle's out_dtype is not used.  Errors as prox_ffn_forward. */
prox_status_t prox_ffn_block_forward(prox_ffn_t* h, const float* x_res_dev, const void* norm_w_dev,
                                     double eps, int B, int k1, int k2, float* x_res_out_dev, void* stream);

/* The FFN sub-blocks of n_layers consecutive layers applied in place to one
 * residual stream (the attention sub-blocks between them are outside the
 * method): one prox_ffn_block_forward per layer, enqueued back to back.
 *   layers     host array of n_layers handles (same d_model)
 *   norm_w     dev bf16 [n_layers, d_model]
 *   x_res      dev fp32 [B, d_model], in and out
 *   trace      NULL, or dev fp32 [n_layers + 1, B, d_model]: the stream before
 *              layer 0 and after every layer (for checking a stack layer by layer)
 * Errors: INVALID_ARG, and those of prox_ffn_block_forward. */
prox_status_t prox_ffn_stack_forward(prox_ffn_t* const* layers, int n_layers, const void* norm_w_dev,
                                     double eps, float* x_res_dev, int B, int k1, int k2,
                                     float* trace_dev_or_null, void* stream);

/* The same two calls with the threshold form of the masks (|x_i| >= tau_x,
 * score_j >= tau_s; per-layer thresholds in host arrays of n_layers floats for
 * the stack).  At B = 1 a layer is one launch; kept counts go to the handle's
 * counters (prox_runtime_sparsity). */
prox_status_t prox_ffn_block_forward_threshold(prox_ffn_t* h, const float* x_res_dev, const void* norm_w_dev,
                                               double eps, int B, float tau_x, float tau_s,
                                               float* x_res_out_dev, void* stream);
prox_status_t prox_ffn_stack_forward_threshold(prox_ffn_t* const* layers, int n_layers, const void* norm_w_dev,
                                               double eps, float* x_res_dev, int B, const float* tau_x_host,
                                               const float* tau_s_host, float* trace_dev_or_null, void* stream);

/* ---- Offline threshold calibration (appendix "Threshold Calibration and Runtime Sparsity", Alg. 1).
 * Host-side state of one (layer, signal) pair: a reservoir of at most `capacity` activation magnitudes
 * (the paper keeps at most 200,000), the threshold "directly from the corresponding empirical quantile",
 * and the saved 4,096-bin histogram.  Not part of the decode hot path: the calls synchronise.
 * Sampling: uniform reservoir (algorithm R); sample number i >= capacity draws
 * j = splitmix64(seed; output i) mod (i + 1) and replaces slot j if j < capacity, so the result is a
 * function of (seed, order of the samples) alone.
 *   prox_calib_add        values_dev: dev bf16 (dtype 0) or fp32 (dtype 1) [n]; |v| is stored as fp32.
 *   prox_calib_threshold  the s-quantile of the reservoir, linear interpolation between order statistics
 *                         (position s (n - 1)), computed in double, returned as the fp32 the kernels
 *                         compare with (|x_i| >= tau_x, score_j >= tau_s).
 *   prox_calib_histogram  counts_host: int64 [4096], equal bins over [0, max]; upper = max magnitude.
 *   prox_calib_seen       samples offered so far / samples held.
 * Errors: INVALID_ARG (NULL, capacity < 1, s outside [0, 1], dtype), NOT_QUANTIZED is not involved,
 * UNSUPPORTED (threshold or histogram of an empty reservoir), CUDA, OOM. */
typedef struct prox_calib prox_calib_t;
prox_status_t prox_calib_create(int64_t capacity, uint64_t seed, prox_calib_t** out);
void prox_calib_destroy(prox_calib_t* c);
prox_status_t prox_calib_add(prox_calib_t* c, const void* values_dev, int64_t n, int dtype, void* stream);
prox_status_t prox_calib_threshold(const prox_calib_t* c, double s, float* tau);
prox_status_t prox_calib_histogram(const prox_calib_t* c, int64_t* counts_host, float* upper);
prox_status_t prox_calib_seen(const prox_calib_t* c, int64_t* seen, int64_t* held);

/* The FFN input of a layer as the block calls form it: xn = bf16(RMSNorm(x_res) * w)
 * (x_res dev fp32 [B, d_model], norm_w dev bf16 [d_model], xn_out dev bf16 [B, d_model]).  Alg. 1
 * collects these as the layer's calibration inputs.  Enqueued on stream.
 * Errors: INVALID_ARG, UNSUPPORTED (B > max_batch), CUDA. */
prox_status_t prox_rmsnorm(prox_ffn_t* h, const float* x_res_dev, const void* norm_w_dev, double eps, int B,
                           void* xn_out_dev, void* stream);

/* Runtime mask counts accumulated by the threshold entry points since the last
 * reset (appendix "Threshold Calibration and Runtime Sparsity":
 * e^ = s2^ - 2 alpha (1 - s1^) / 3).  Host-synchronous.  Any pointer may be NULL. */
prox_status_t prox_runtime_sparsity(prox_ffn_t* h, double alpha, int64_t* tokens,
                                    double* s1_hat, double* s2_hat, double* e_hat, int reset);

/* Budget helper (Sec. 4.2): s2 = s_ref, s1 from e = s2 - 2 alpha (1 - s1) / 3;
 * if s1 leaves [s1_min, s1_max] it is clamped and s2 re-solved.  Host only. */
prox_status_t prox_allocate_budget(double e, double alpha, double s_ref, double s1_min,
                                   double s1_max, double* s1, double* s2);

/* k = clamp(floor((1 - s) * dim + 0.5), 1, dim).  Host only. */
prox_status_t prox_sparsity_to_k(double s, int dim, int* k);

/* Test hook: unpack the stored proxy of W_gate (which = 0) or W_up (1) into
 * host q int8 [F, D] and host scale fp32 [F, D/group] (group = D if per-row).
 * Synchronises.  Errors: INVALID_ARG, NOT_QUANTIZED, CUDA, OOM. */
prox_status_t prox_proxy_export(prox_ffn_t* h, int which, int8_t* q_host, float* scale_host);

/* Test hook: the Stage-1 input mask alone.  idx dev int32 [B, k1], ascending. */
prox_status_t prox_input_topk(prox_ffn_t* h, const void* x_dev, int B, int k1,
                              int32_t* idx_dev, void* stream);

/* Offline packer output: write / read the packed proxies, scales and the
 * channel-major W_down of a quantized handle.  prox_pack_load needs a handle
 * created over the same weights and shape; it replaces prox_quantize_proxy.
 * Both synchronise.  Errors: INVALID_ARG, NOT_QUANTIZED, IO, CUDA, OOM. */
prox_status_t prox_pack_save(prox_ffn_t* h, const char* path);
prox_status_t prox_pack_load(prox_ffn_t* h, const char* path, void* stream);

/* Bytes the method must move for one call at these budgets (B = 1 layout,
 * `rows_in` kept input rows and `rows_ch` kept channel rows actually read):
 * proxy rows + scales + gate/up rows + down rows + activations.  Host only. */
prox_status_t prox_algorithmic_bytes(const prox_ffn_t* h, int rows_in, int rows_ch,
                                     int64_t* stage1, int64_t* gate_up, int64_t* down,
                                     int64_t* activations);

/* Device-side diagnostics: 0 if no kernel recorded a problem since the last
 * read; otherwise a bit set (1 = channel id out of range skipped, 2 = input id
 * out of range skipped, 4 = bounded wait expired).  Reading clears it.
 * Synchronises the given stream.  If bit 4 is set the call that ran into the wait
 * did not write its output (y is undefined); the handle's shared counters are put
 * back to their idle state here and the call returns PROX_ERR_TIMEOUT (with *code
 * filled in); the next forward call is an ordinary one.  prox_ffn_forward_host,
 * which synchronises anyway, checks for an expired wait itself and returns
 * PROX_ERR_TIMEOUT in the same way. */
prox_status_t prox_last_device_status(prox_ffn_t* h, int32_t* code, void* stream);

/* Per-kernel timing hook for benchmarks.  While enabled, every kernel launched
 * through the handle is bracketed by CUDA events on the call's stream (this
 * adds event records to the stream and must not be on during stream capture).
 * prox_profile_read synchronises those events, adds up launches and
 * milliseconds per kernel kind into counts[PROX_NUM_KERNEL_KINDS] and
 * ms[PROX_NUM_KERNEL_KINDS] (host arrays), and forgets them.  Kinds, in order:
 * input_select, proxy_gemv, channel_select, gateup, down, finalize, fused, union. */
#define PROX_NUM_KERNEL_KINDS 8
prox_status_t prox_profile_enable(prox_ffn_t* h, int on);
prox_status_t prox_profile_read(prox_ffn_t* h, int64_t* counts_host, double* ms_host);

/* Number of kernels this library launched through the handle so far. */
prox_status_t prox_launch_count(const prox_ffn_t* h, int64_t* launches);

void prox_ffn_destroy(prox_ffn_t* h);
const char* prox_status_string(prox_status_t s);
/* Text of the CUDA error behind the calling thread's most recent PROX_ERR_CUDA /
 * PROX_ERR_OOM ("" if none). */
const char* prox_last_cuda_error(void);
const char* prox_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PROX_H_ */
