/*
 * qzo.h - C ABI of the QZO hot path on NVIDIA B200 (sm_100a).
 *
 * QZO (Quantized Zeroth-order Optimization) fine-tunes a weight-only int4 LLM by
 * perturbing only its quantisation scales.  One optimisation step (Algorithm 1) is
 *   l+ = L((Delta + eps z) (.) theta_bar; B)          first forward
 *   l- = L((Delta - eps z) (.) theta_bar; B)          second forward
 *   d  = (l+ - l-) / (2 eps),  d' = clip(d, -C, C)    Eq. 5, Eq. 6
 *   Delta_i <- max(Delta_i - eta d' z_i, 0)           seeded update
 * with z ~ N(0, I) regenerated from a seed and never stored (Sec. 3.1).
 *
 * Conventions
 *  - Every pointer named d_* is a DEVICE pointer owned by the caller; h_* is a HOST
 *    pointer.  The library allocates no device memory: model state lives in the
 *    caller's tensors and in one caller-provided workspace.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Calls are asynchronous on that stream unless stated otherwise.
 *  - Every function returns QZO_OK (0) or a negative qzo_status.  No exceptions cross
 *    the boundary.  A model handle must not be used from two threads at once.
 *  - Only compute-capability 10.x devices are supported; there is no CPU or other
 *    backend (QZO_ERR_UNSUPPORTED_DEVICE).
 *
 * Interchange layouts
 *  - int4 weights, logical q[k][n] in [-8, 7] for Y[t][n] = sum_k X[t][k] W[k][n]:
 *    uint32 [K/8][N] row-major, nibble j (bits 4j..4j+3) of word [kw][n] holds
 *    u = q[8 kw + j][n] + 8.  K must be a multiple of 8, N a multiple of 8.
 *  - scales: bf16 [G][N] row-major, G = ceil(K / 128); group g covers rows
 *    128 g .. 128 g + 127 (Eq. 3, Eq. 4 with the group of 128 the paper uses).
 *  - logical scale index of scale [g][n] of a linear: index_base + g N + n.  It selects
 *    the Gaussian z_i = z(seed, i) (Philox4x32-10, see qzo_normals) and is independent of
 *    any tiling.  index_base must be a multiple of 4.
 *  - kernel layout of the int4 weights: produced by qzo_repack_int4; opaque.
 */
#ifndef QZO_H_
#define QZO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QZO_OK = 0,
  QZO_ERR_BAD_ARG = -1,            /* null pointer, bad size, sign not in {-1,0,1}, eps <= 0, clip < 0 ... */
  QZO_ERR_UNSUPPORTED_DEVICE = -2, /* current device is not sm_100 */
  QZO_ERR_WORKSPACE = -3,          /* workspace too small or misaligned (256 bytes) */
  QZO_ERR_NONFINITE = -4,          /* a loss or g is NaN/Inf; scales were left untouched */
  QZO_ERR_DEVICE_TIMEOUT = -5,     /* a bounded device-side wait expired (status word); scales untouched by that step */
  QZO_ERR_CUDA = -6,               /* a CUDA call failed; see qzo_last_cuda_error */
  QZO_ERR_MISSING_TENSOR = -7      /* qzo_init_model: a required tensor was not supplied */
} qzo_status;

enum { QZO_ARCH_LLAMA = 0, QZO_ARCH_OPT = 1 };
enum { QZO_DTYPE_BF16 = 0, QZO_DTYPE_F32 = 1, QZO_DTYPE_U32 = 2, QZO_DTYPE_I32 = 3 };

/* Human-readable text of a status code (static storage). */
const char* qzo_strerror(int status);
/* cudaError_t value of the last failed CUDA call in this process (0 if none). */
int qzo_last_cuda_error(void);

/* ------------------------------------------------------------------------------------
 * Building blocks (each is one step of the path; exported for parity tests and sweeps)
 * ---------------------------------------------------------------------------------- */

/* Philox4x32-10 words of counter blocks block_base .. block_base+n_blocks-1 under key
 * `seed` (Sec. 3.1: only the seed is stored).  d_words: uint32 [n_blocks][4].
 * d_uniforms (may be NULL): float [n_blocks][4], U(x) = ((x >> 9) + 0.5) 2^-23. */
int qzo_philox_words(uint64_t seed, uint64_t block_base, int64_t n_blocks,
                     uint32_t* d_words, float* d_uniforms, void* stream);

/* z_i for i = index_base .. index_base+count-1 (Algorithm 1: "z ~ N(0,1)" after the
 * generator is reset with seed s).  d_z: float [count]. */
int qzo_normals(uint64_t seed, uint64_t index_base, int64_t count, float* d_z, void* stream);

/* Eq. 3 with Delta = absmax / (2^(4-1) - 1) per group of 128 rows and per column:
 * d_w float [K][N] -> d_qpacked uint32 [K/8][N] (interchange), d_scales bf16 [G][N].
 * Scale = bf16(absmax/7); q = clamp(rne(w / scale), -8, 7); zero scale gives q = 0. */
int qzo_quantize_int4(const float* d_w, int K, int N, uint32_t* d_qpacked, void* d_scales_bf16,
                      void* stream);

/* Eq. 4 storage: interchange uint32 [K/8][N] -> int8 q [K][N] (for bit-exact checks). */
int qzo_unpack_int4(const uint32_t* d_qpacked, int K, int N, int8_t* d_q, void* stream);

/* Size in bytes of the kernel-layout copy of a K x N int4 weight. */
int qzo_repacked_bytes(int K, int N, size_t* bytes);
/* interchange -> kernel layout (done once; theta_bar is fixed for the whole run,
 * the integer weights that Algorithm 1 takes as an input).  d_out: `bytes` from qzo_repacked_bytes, 256-aligned. */
int qzo_repack_int4(const uint32_t* d_qpacked, int K, int N, void* d_out, size_t out_bytes,
                    void* stream);
/* kernel layout -> int8 q [K][N]: what the GEMM's prologue sees (bit-exact check). */
int qzo_unpack_kernel_layout(const void* d_wq, int K, int N, int8_t* d_q, void* stream);

/* Workspace the GEMM needs for a problem (0 if none; split-K partial sums otherwise). */
int qzo_gemm_workspace_bytes(int M, int K, int N, size_t* bytes);

/* Perturbed W4A16 linear (Eq. 4 inside Eq. 5):
 *   Y[t][n] = sum_k X[t][k] (s[k/128][n] + sign eps z_i) q[k][n] (+ bias[n]),
 *   i = scale_index_base + (k/128) N + n; the perturbed scale is formed in fp32 inside the
 *   de-quantisation prologue; the stored scales are never modified.
 * d_x bf16 [M][K] row-major; d_wq kernel layout (qzo_repack_int4); d_scales bf16 [G][N];
 * d_bias float [N] or NULL; d_y bf16 [M][N], 16-byte aligned.  sign in {-1, 0, +1} (0 = unperturbed).
 * d_workspace: qzo_gemm_workspace_bytes, 256-aligned (may be NULL when that is 0).
 * d_status: int on the device, set non-zero if a bounded wait expired (may be NULL). */
int qzo_perturbed_gemm(const void* d_x_bf16, const void* d_wq, const void* d_scales_bf16,
                       const float* d_bias, void* d_y_bf16, int M, int K, int N,
                       uint64_t seed, uint64_t scale_index_base, int sign, float eps,
                       void* d_workspace, size_t workspace_bytes, int* d_status, void* stream);

/* The same linear for weights stored as 4-bit codes into a 16-entry table with one scale per block of 64
 * rows (block-scaled codebook storage such as NF4; the paper applies QZO to NF4 weights in its appendix
 * "Results with Stable Diffusion" and to codebook weights with channel-wise scales in Sec. 4.1: what QZO
 * perturbs and updates is the format's continuous scale, Eq. 5, so only the de-quantisation prologue differs):
 *   Y[t][n] = sum_k X[t][k] (s[k/64][n] + sign eps z_i) table[c[k][n]] (+ bias[n]),  i = scale_index_base + (k/64) N + n.
 * d_codes: codes c in [0, 15] in the kernel layout of qzo_repack_int4 (pack them like int4 values, code =
 * stored nibble); d_scales bf16 [ceil(K/64)][N]; h_table16: HOST pointer to the 16 table values (read during
 * the call, rounded to bf16 on the device).  Everything else as qzo_perturbed_gemm; the seeded update of such
 * scales is qzo_update_scales_flat. */
int qzo_perturbed_gemm_table16(const void* d_x_bf16, const void* d_codes, const void* d_scales_bf16,
                               const float* h_table16, const float* d_bias, void* d_y_bf16, int M, int K, int N,
                               uint64_t seed, uint64_t scale_index_base, int sign, float eps,
                               void* d_workspace, size_t workspace_bytes, int* d_status, void* stream);

/* The same table prologue for weights whose only continuous parameter is one scale per OUTPUT CHANNEL (the
 * paper's codebook setting, Sec. 4.1: AQLM-style codebook weights, of which QZO tunes the channel-wise scales;
 * here with a 16-entry scalar table standing in for the codebook):
 *   Y[t][n] = (s[n] + sign eps z_i) sum_k X[t][k] table[c[k][n]] (+ bias[n]),  i = scale_index_base + n.
 * d_scales bf16 [N]; everything else as qzo_perturbed_gemm_table16.  The seeded update of such scales is
 * qzo_update_scales_flat over N entries. */
int qzo_perturbed_gemm_codebook16_channelwise(const void* d_x_bf16, const void* d_codes, const void* d_scales_bf16,
                                              const float* h_table16, const float* d_bias, void* d_y_bf16,
                                              int M, int K, int N, uint64_t seed, uint64_t scale_index_base,
                                              int sign, float eps, void* d_workspace, size_t workspace_bytes,
                                              int* d_status, void* stream);

/* The same linear for callers that must not allocate device memory and have no workspace to
 * lend: for example a serving process that gave all device memory to its own pool when it
 * started, or a latency-critical loop in which the device-wide synchronisation of an allocation
 * is not acceptable.  (The paper has no counterpart; this is a property of the library.)
 * Arguments and result are those of qzo_perturbed_gemm without the workspace.  The split-K
 * partial sums go to a fixed array of QZO_NOALLOC_SCRATCH_BYTES inside the library image: every
 * device that loads the library holds that much until the process exits.  The call allocates
 * nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *  - A problem whose partial sums (qzo_gemm_workspace_bytes) exceed the array returns
 *    QZO_ERR_WORKSPACE and launches nothing.
 *  - The first call on each device looks the array's device address up (with that device
 *    current).  If no kernel of the library has run on that device yet, this is also the moment the
 *    driver loads the library's device code and reserves the array, which may synchronise the device:
 *    make that first call at start-up, and before any stream capture begins.  Later calls do neither.
 *  - All calls on a device share the one array, which keeps the last call's partial sums (none
 *    of it needs clearing: each call overwrites every element it later reads).  Two calls that
 *    overlap on the GPU (different streams) race on it; keep them on one stream or order them. */
#define QZO_NOALLOC_SCRATCH_BYTES (16u << 20)
int qzo_perturbed_gemm_noalloc(const void* d_x_bf16, const void* d_wq, const void* d_scales_bf16,
                               const float* d_bias, void* d_y_bf16, int M, int K, int N,
                               uint64_t seed, uint64_t scale_index_base, int sign, float eps,
                               int* d_status, void* stream);

/* Seeded update of a flat run of scales (Algorithm 1, last loop, with Eq. 6 applied to g):
 *   s_i <- bf16(max(s_i - (lr clip(g,-C,C)) z_i, 0)), i = index_base .. index_base+count-1.
 * d_scales bf16 [count], in place.  g must be finite, clip >= 0. */
int qzo_update_scales_flat(void* d_scales_bf16, int64_t count, uint64_t seed, uint64_t index_base,
                           float lr, float g, float clip, void* stream);

/* ------------------------------------------------------------------------------------
 * Model-level entry points
 * ---------------------------------------------------------------------------------- */

typedef struct qzo_model qzo_model; /* opaque handle (host memory owned by the library) */

typedef struct {
  int arch;        /* QZO_ARCH_LLAMA: RMSNorm, RoPE, SiLU-gated MLP, no bias;
                      QZO_ARCH_OPT: LayerNorm, learned positions, ReLU MLP, biases */
  int n_layers, d_model, n_heads, d_ffn, vocab, max_seq;
  int group_size;  /* must be 128 */
  float norm_eps, rope_theta;
} qzo_model_desc;

typedef struct {
  const char* name; /* see qzo_init_model */
  void* dptr;       /* device pointer */
  int dtype;        /* QZO_DTYPE_* */
  int64_t shape[2]; /* rows, cols (cols = 1 for vectors) */
} qzo_tensor;

/* Number of entries of the flat scale buffer (all block linears, layer-major, in the order
 * q,k,v,o,gate,up,down (Llama) / q,k,v,o,fc1,fc2 (OPT), each base rounded up to a multiple
 * of 8) and the number of trainable scales (Table 2: block linear weights / 128). */
int qzo_num_scales(const qzo_model_desc* desc, int64_t* flat_entries, int64_t* trainable);
/* Where linear `linear` (position in the order above) of layer `layer` sits in the flat buffer. */
int qzo_scale_layout(const qzo_model_desc* desc, int layer, int linear,
                     int64_t* index_base, int* G, int* N);

/* Bytes of workspace qzo_init_model needs for batches up to max_tokens = B*S tokens
 * (kernel-layout weights + activations + fp32 logits + split-K partials).  The activation
 * buffers hold 2 * max_tokens rows, because qzo_step runs both passes as one forward. */
int qzo_workspace_bytes(const qzo_model_desc* desc, int max_tokens, size_t* bytes);

/* Binds a model to caller-owned tensors (the inputs of Algorithm 1: scales Delta, integer
 * weights theta_bar).  Tensors, by name:
 *   "embed" bf16 [V][d]; "lm_head" bf16 [V][d]; "pos_embed" bf16 [max_seq][d] (OPT);
 *   "final_norm_w" f32 [d] (+ "final_norm_b", OPT); "scales" bf16 [flat_entries] (trained in place);
 *   "L<i>.norm1_w", "L<i>.norm2_w" f32 [d] (+ "_b", OPT);
 *   "L<i>.<lin>.qweight" u32 [K/8][N] interchange layout (copied into the workspace in kernel
 *   layout during this call; the caller may free it after the stream has drained);
 *   "L<i>.<lin>.bias" f32 [N] (OPT).
 * d_workspace: qzo_workspace_bytes, 256-aligned, must outlive the handle. */
int qzo_init_model(const qzo_model_desc* desc, const qzo_tensor* tensors, int n_tensors,
                   void* d_workspace, size_t workspace_bytes, int max_tokens, void* stream,
                   qzo_model** out);
int qzo_free_model(qzo_model* m);

/* One forward pass, L(Delta' (.) theta_bar; B) with Delta' = Delta + sign eps z(seed)
 * (either forward pass of Algorithm 1; sign 0 = unperturbed).  d_tokens, d_labels:
 * int32 [B][S]; label -100 is ignored; loss = mean next-token cross entropy over kept
 * positions, written to d_loss (float, device). */
int qzo_forward_loss(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S,
                     uint64_t seed, int sign, float eps, float* d_loss);

/* Seeded update of every scale of the model with a host-side g (clipped here, Eq. 6).
 * Non-finite g: QZO_ERR_NONFINITE and no write. */
int qzo_update_scales(qzo_model* m, uint64_t seed, float lr, float g, float clip);

/* Whole step of Algorithm 1 on device-resident tokens: two forwards (sign +1, -1), d, d' and
 * the update, with d formed on the device.  When B*S is 16, 32, 64, 128 or a multiple of 256 the
 * two forwards run as ONE pass over two copies of the batch (rows of the second copy take
 * -eps z); every kernel works row by row or sequence by sequence, so the losses are the ones two
 * separate passes give, bit for bit.
 * From the second call with the same (B, S) on, the launch sequence of the two forwards is replayed from a CUDA
 * graph recorded once (its GEMMs read seed and eps from device memory, the tokens come from the model's own
 * buffers); results are bit-identical to the direct launches.  See qzo_use_recorded_steps.
 * h_out (may be NULL): {l+, l-, d, d'}; when
 * non-NULL the call synchronises the stream.  The scales are left untouched (the update coefficient is
 * forced to zero on the device) and, when h_out is given, an error is returned if
 *  - either loss is not finite: QZO_ERR_NONFINITE;
 *  - a bounded device-side wait expired in any launch since qzo_init_model: QZO_ERR_DEVICE_TIMEOUT;
 *  - a token id lies outside [0, vocab): QZO_ERR_BAD_ARG.
 * The last two are sticky (status word, see qzo_device_status). */
int qzo_step(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S,
             uint64_t seed, float eps, float lr, float clip, float* h_out);

/* Recorded steps (CUDA graphs) of qzo_step / qzo_step_host / qzo_step_begin: on != 0 (the default) allows them, 0 makes every
 * step issue its launches directly.  They are bypassed anyway while joint mode, a debug capture or the per-GEMM
 * timing is on, for batch shapes beyond the first 16 a model has seen, and switched off for good if recording
 * ever fails. */
int qzo_use_recorded_steps(qzo_model* m, int on);
/* *h_count = number of batch shapes whose step is recorded at the moment, or -1 when recorded steps are
 * switched off (by qzo_use_recorded_steps, or because recording failed). */
int qzo_recorded_step_count(qzo_model* m, int* h_count);

/* The two halves of qzo_step, for data-parallel replicas (every rank holds the same theta_bar and Delta
 * and its own part of the batch; z depends on (seed, index) only, Sec. 3.1, so ranks exchange losses,
 * never parameters).
 * qzo_step_begin runs the two forward passes of Algorithm 1 on this rank's tokens and writes
 *   d_sums (device, float[4], 16-byte aligned) = {sum of token losses with +eps z, the same with -eps z,
 *   kept tokens of the + pass, kept tokens of the - pass}.
 * Between the calls the caller may add the d_sums of all ranks element by element (one all-reduce of four
 * floats, asynchronously on the same stream).  qzo_step_finish then forms l+- = sum / count, d = (l+ - l-) /
 * (2 eps), d' = clip(d, -C, C) (Eq. 6) and applies the seeded update (Algorithm 1, last loop), all on the
 * device; given equal d_sums and seed every rank ends with bit-identical scales.  h_out and the error
 * behaviour are those of qzo_step.  qzo_step is qzo_step_begin followed by qzo_step_finish. */
int qzo_step_begin(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S,
                   uint64_t seed, float eps, float* d_sums);
int qzo_step_finish(qzo_model* m, const float* d_sums, uint64_t seed, float eps, float lr, float clip,
                    float* h_out);

/* Joint mode (Sec. 3.2.1, closing remark: Q-SPSA on the scales may be combined with SPSA on the
 * un-quantised parts; Sec. 4.1, implementation details: the experiments with codebook weights train the
 * un-quantised parts that way, with plain SPSA and ZO-SGD).
 * After qzo_enable_joint_spsa every perturbed forward (sign +1 / -1) also perturbs the embedding matrix, the
 * lm_head matrix and every norm gain (and norm bias, OPT) as theta + sign eps z (Def. 3.1), and every step
 * also updates them in place, theta <- theta - lr_dense d' z (Def. 3.2; no clamp, that belongs to the
 * scales), with the same clipped d' as the scales.  z comes from the same (seed, index) stream at indices
 * that follow the scales': each base rounded up to a multiple of 8, in the order embed, lm_head, then per
 * layer norm1 gain (bias), norm2 gain (bias), then the final norm.  Position embeddings and the biases of
 * the linears stay fixed.  The caller's "embed", "lm_head" and norm tensors must be writable.
 * d_workspace: qzo_joint_workspace_bytes (perturbed copies of the vectors and of the lm_head for both
 * signs), 256-aligned, must outlive the handle; NULL switches the mode off.  Synchronises the stream. */
int qzo_joint_workspace_bytes(const qzo_model_desc* desc, size_t* bytes);
int qzo_enable_joint_spsa(qzo_model* m, void* d_workspace, size_t workspace_bytes, float lr_dense);

/* Same step with HOST token / label buffers (int32 [B][S]); copies them in, runs the step and
 * reads {l+, l-, d, d'} back.  Synchronises. */
int qzo_step_host(qzo_model* m, const int32_t* h_tokens, const int32_t* h_labels, int B, int S,
                  uint64_t seed, float eps, float lr, float clip, float* h_out);

/* The trainable state (the inputs of Algorithm 1: the quantisation scales Delta that the caller hands over
 * and gets back).  linear_id = layer * L + position, L = 7 (Llama: q,k,v,o,gate,up,down) or 6 (OPT:
 * q,k,v,o,fc1,fc2): copies that linear's bf16 [G][N] scales out of / into the model's flat buffer;
 * linear_id = -1: the whole flat buffer (qzo_num_scales entries).  d_bf16 is a device pointer; `bytes` must
 * be exactly the size of what is copied (QZO_ERR_BAD_ARG otherwise).  Asynchronous on the model's stream.
 * Because z is a function of (seed, index) only, scales + step counter + base seed resume a run exactly. */
int qzo_get_scales(qzo_model* m, int linear_id, void* d_bf16, size_t bytes);
int qzo_set_scales(qzo_model* m, int linear_id, const void* d_bf16, size_t bytes);

/* Selects the decoder block whose output later forwards keep a copy of (-1 = none). */
int qzo_debug_set_capture(qzo_model* m, int layer);
/* Copies an intermediate of the LAST forward into d_out (bf16 [T][d] for which = 0: output of
 * decoder block `layer`, which must be the block chosen with qzo_debug_set_capture before that
 * forward; float [T][V] for which = 1: logits, layer ignored).  T is the token count of that
 * forward: B*S after qzo_forward_loss, 2*B*S after a qzo_step that ran both signs as one pass
 * (rows of the sign +1 copy first).  bytes below the size needed: QZO_ERR_BAD_ARG. */
int qzo_debug_layer_output(qzo_model* m, int layer, int which, void* d_out, size_t bytes);

/* Test entry for the bounded device-side waits (failure detection without a fault): runs the perturbed GEMM
 * (seed 1, sign +1, eps 1e-3, no bias, a problem without split-K) with the copies of quantisation group
 * `skip_group` of every CTA announced but never issued and with every wait bounded by wait_limit_cycles
 * (capped at the normal limit of about two seconds).  Every role of the kernel then runs out of its wait,
 * the CTA drains the copies it did issue, frees its tensor memory and RETURNS; *d_status becomes non-zero.
 * Nothing traps and nothing spins without bound.  The output is unspecified.  Later calls are unaffected. */
int qzo_debug_gemm_wait_expiry(const void* d_x_bf16, const void* d_wq, const void* d_scales_bf16, void* d_y_bf16,
                               int M, int K, int N, int skip_group, int64_t wait_limit_cycles, int* d_status,
                               void* stream);

/* Reads the device status word: bit 0 = a bounded device-side wait expired in some launch since init
 * (returns QZO_ERR_DEVICE_TIMEOUT), bit 1 = a token id outside [0, vocab) was seen (QZO_ERR_BAD_ARG);
 * 0 = nothing to report.  Synchronises. */
int qzo_device_status(qzo_model* m, int* h_status);
/* Overwrites the status word from the host (0 clears it).  For tests of the error path of a step and
 * for clearing the word after the caller has dealt with a report.  Synchronises. */
int qzo_debug_set_status(qzo_model* m, int value);

/* Per-GEMM timing: with max_launches > 0 every later perturbed-GEMM launch of this model (up to
 * max_launches between two reads) is bracketed by a pair of CUDA events on the model's stream;
 * 0 switches it off.  qzo_profile_read synchronises, returns the number of bracketed launches,
 * the sum of their durations in ms and of their algorithmic FLOPs (2 M K N), and rearms. */
int qzo_profile_gemms(qzo_model* m, int max_launches);
int qzo_profile_read(qzo_model* m, int64_t* launches, double* total_ms, double* total_flops);

/* Number of kernels the library launched since the process started, those of replayed recorded steps
 * included (for benchmark accounting). */
int64_t qzo_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* QZO_H_ */
