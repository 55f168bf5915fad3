// Host orchestration of the model-level entry points: binds caller-owned tensors, lays the
// workspace out, and issues the launch sequence of one forward pass and of one QZO step
// (Algorithm 1) on the caller's stream.  No device memory is allocated here.
#include "qzo_common.cuh"
#include "launch.cuh"
#include "layers.cuh"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <vector>

namespace qzo {

static std::atomic<int> g_last_cuda_error{0};
static std::atomic<long long> g_launches{0};
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error.store((int)e); }
int last_cuda_error() { return g_last_cuda_error.load(); }
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
void add_launches(long long n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
long long launch_count() { return g_launches.load(); }

int check_device() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { set_last_cuda_error(e); return QZO_ERR_UNSUPPORTED_DEVICE; }
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) { set_last_cuda_error(e); return QZO_ERR_UNSUPPORTED_DEVICE; }
  return major == 10 ? QZO_OK : QZO_ERR_UNSUPPORTED_DEVICE;
}

struct LinearShape { const char* name; int K, N; };

static int linear_shapes(const qzo_model_desc& d, LinearShape out[7]) {
  const int dm = d.d_model, f = d.d_ffn;
  if (d.arch == QZO_ARCH_LLAMA) {
    const LinearShape s[7] = {{"q", dm, dm}, {"k", dm, dm}, {"v", dm, dm}, {"o", dm, dm},
                              {"gate", dm, f}, {"up", dm, f}, {"down", f, dm}};
    memcpy(out, s, sizeof(s));
    return 7;
  }
  const LinearShape s[6] = {{"q", dm, dm}, {"k", dm, dm}, {"v", dm, dm}, {"o", dm, dm}, {"fc1", dm, f}, {"fc2", f, dm}};
  memcpy(out, s, sizeof(s));
  return 6;
}

int validate_desc(const qzo_model_desc* d) {
  if (!d) return QZO_ERR_BAD_ARG;
  if (d->arch != QZO_ARCH_LLAMA && d->arch != QZO_ARCH_OPT) return QZO_ERR_BAD_ARG;
  if (d->n_layers <= 0 || d->d_model <= 0 || d->n_heads <= 0 || d->d_ffn <= 0 || d->vocab <= 0 || d->max_seq <= 0)
    return QZO_ERR_BAD_ARG;
  if (d->group_size != kGroup) return QZO_ERR_BAD_ARG;
  if (d->d_model % d->n_heads) return QZO_ERR_BAD_ARG;
  const int dh = d->d_model / d->n_heads;
  if (dh != 64 && dh != 128) return QZO_ERR_BAD_ARG;
  if ((d->d_model % 8) || (d->d_ffn % 8)) return QZO_ERR_BAD_ARG;
  if (!(d->norm_eps > 0.0f)) return QZO_ERR_BAD_ARG;
  if (d->arch == QZO_ARCH_LLAMA && !(d->rope_theta > 0.0f)) return QZO_ERR_BAD_ARG;
  return QZO_OK;
}

// Index base of (layer, linear) and running total, bases rounded up to a multiple of 8.
int64_t scale_layout(const qzo_model_desc& d, int layer, int linear, int* G, int* N, int64_t* trainable) {
  LinearShape ls[7];
  const int nl = linear_shapes(d, ls);
  int64_t run = 0, train = 0, found = -1;
  for (int L = 0; L < d.n_layers; ++L) {
    for (int i = 0; i < nl; ++i) {
      run = (run + 7) / 8 * 8;
      const int g = ceil_div(ls[i].K, kGroup);
      if (L == layer && i == linear) {
        found = run;
        if (G) *G = g;
        if (N) *N = ls[i].N;
      }
      run += (int64_t)g * ls[i].N;
      train += (int64_t)g * ls[i].N;
    }
  }
  if (trainable) *trainable = train;
  return (layer < 0) ? run : found;
}

struct Linear {
  int K = 0, N = 0;
  int64_t idx_base = 0;
  const void* wq = nullptr;     // kernel layout, inside the workspace
  const float* bias = nullptr;
};
struct Layer {
  const float *norm1_w = nullptr, *norm1_b = nullptr, *norm2_w = nullptr, *norm2_b = nullptr;
  Linear lin[7];
};

}  // namespace qzo

struct qzo_model {
  qzo_model_desc desc;
  int n_lin = 0;
  std::vector<qzo::Layer> layers;
  const __nv_bfloat16 *embed = nullptr, *lm_head = nullptr, *pos_embed = nullptr;
  const float *final_norm_w = nullptr, *final_norm_b = nullptr;
  __nv_bfloat16* scales = nullptr;
  int64_t flat_entries = 0;
  int max_tokens = 0;
  cudaStream_t stream = nullptr;
  // workspace regions
  __nv_bfloat16 *x = nullptr, *xn = nullptr, *qkv = nullptr, *att = nullptr, *mlp_a = nullptr, *mlp_b = nullptr,
                *capture = nullptr;
  float *logits = nullptr, *row_loss = nullptr, *loss2 = nullptr, *sums = nullptr, *out7 = nullptr, *rope_cs = nullptr;
  int32_t *tok_dev = nullptr, *lab_dev = nullptr;
  void* gemm_ws = nullptr;
  size_t gemm_ws_bytes = 0;
  int* status = nullptr;
  int capture_layer = -1;
  int last_T = 0;
  // joint mode (plain SPSA on the un-quantised tensors), off unless qzo_enable_joint_spsa was called
  bool joint = false;
  float lr_dense = 0.0f;
  int n_vec = 0;                              // norm gain / bias vectors, in the order of the index ranges
  int64_t base_embed = 0, base_lm_head = 0;   // logical indices of the two matrices
  const float* const* vec_table = nullptr;    // device: pointers to the vectors
  const unsigned long long* vec_base = nullptr;   // device: their logical index bases
  float *vec_plus = nullptr, *vec_minus = nullptr;   // perturbed copies [n_vec][d]
  __nv_bfloat16 *lm_plus = nullptr, *lm_minus = nullptr;   // perturbed copies of the lm_head [V][d]
  // recorded steps: one CUDA graph per (B, S) holding a step's two forwards; its GEMMs read seed and eps from sp_dev
  struct RecordedStep {
    cudaGraphExec_t exec = nullptr;
    long long launches = 0;                   // kernels of one replay
    int rows = 0;                             // token rows of the step's forward (what last_T is after it)
    bool seen = false;                        // the shape ran once the direct way (per-device set-up done)
  };
  bool use_graphs = true;
  std::map<long long, RecordedStep> recorded;
  cudaStream_t rec_stream = nullptr;          // recording only; nothing ever runs on it
  qzo::StepParams* sp_dev = nullptr;
  const qzo::StepParams* cur_sp = nullptr;    // non-null while a step is being recorded
  // optional per-GEMM timing (CUDA events around every perturbed GEMM launch)
  bool profiling = false;
  std::vector<cudaEvent_t> events;
  size_t events_used = 0;
  double profiled_flops = 0.0;
};

namespace qzo {

struct WsPlan {
  size_t off_weights, off_x, off_xn, off_qkv, off_att, off_a, off_b, off_capture, off_logits, off_rowloss, off_scalars,
      off_rope, off_tok, off_lab, off_gemm, gemm_bytes, total;
};

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Activation buffers hold twice the caller's token limit: a step runs its two passes (perturbation
// signs +1 and -1) as one forward over both copies of the batch.
int plan_workspace(const qzo_model_desc& d, int max_tokens, WsPlan* p) {
  const int T = 2 * max_tokens;
  LinearShape ls[7];
  const int nl = linear_shapes(d, ls);
  size_t off = 0;
  p->off_weights = off;
  size_t per_layer = 0;
  for (int i = 0; i < nl; ++i) per_layer += align_up(repacked_bytes(ls[i].K, ls[i].N), 256);
  off += per_layer * d.n_layers;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t dm = d.d_model, f = d.d_ffn;
  p->off_x = take((size_t)T * dm * 2);
  p->off_xn = take((size_t)T * dm * 2);
  p->off_qkv = take((size_t)T * 3 * dm * 2);
  p->off_att = take((size_t)T * dm * 2);
  p->off_a = take((size_t)T * f * 2);
  p->off_b = take((size_t)T * f * 2);
  p->off_capture = take((size_t)T * dm * 2);
  p->off_logits = take((size_t)T * d.vocab * 4);
  p->off_rowloss = take((size_t)T * 4);
  p->off_scalars = take(64 * 4);
  p->off_rope = take((size_t)d.max_seq * (dm / d.n_heads) * 4);
  p->off_tok = take((size_t)T * 4);
  p->off_lab = take((size_t)T * 4);
  // split-K partial sums: the largest need over every token count a launch of this model can have
  // (any B*S up to max_tokens in a single-sign pass, twice that in a paired step); only token counts
  // up to the largest split token tile can split, the rest is covered by the two limits themselves
  size_t gb = 0;
  for (int i = 0; i < nl; ++i) {
    for (int M = 1; M <= std::min(T, kMaxSplitTokens); ++M) gb = std::max(gb, gemm_workspace_bytes(M, ls[i].K, ls[i].N));
    for (int half = 16; half <= std::min(max_tokens, kMaxSplitTokens); half *= 2)      // paired steps of few tokens
      gb = std::max(gb, gemm_workspace_bytes(2 * half, ls[i].K, ls[i].N, half));
    gb = std::max(gb, std::max(gemm_workspace_bytes(T, ls[i].K, ls[i].N), gemm_workspace_bytes(max_tokens, ls[i].K, ls[i].N)));
  }
  p->gemm_bytes = gb;
  p->off_gemm = take(gb);
  p->total = off;
  return QZO_OK;
}

// x += delta (when delta is given), then out = norm(x): the residual add of a block's projection is
// fused into the norm that follows it.
// vec: position of the gain among the joint mode's vectors (its bias, if any, follows it); sign and
// pair_rows say which perturbed copy a row takes in joint mode (sign 0: the stored vectors).
static int add_norm(qzo_model* m, __nv_bfloat16* x, const __nv_bfloat16* delta, const float* w, const float* b, int vec,
                    int sign, int pair_rows, int T, __nv_bfloat16* out) {
  const float *w2 = nullptr, *b2 = nullptr;
  int pr = 0;
  if (m->joint && sign != 0) {
    const size_t d = m->desc.d_model;
    const float* first = sign > 0 ? m->vec_plus : m->vec_minus;
    const float* second = sign > 0 ? m->vec_minus : m->vec_plus;
    w = first + (size_t)vec * d;
    if (b) b = first + (size_t)(vec + 1) * d;
    if (pair_rows > 0) {
      pr = pair_rows;
      w2 = second + (size_t)vec * d;
      if (b) b2 = second + (size_t)(vec + 1) * d;
    }
  }
  if (m->desc.arch == QZO_ARCH_LLAMA)
    return launch_add_rmsnorm(x, delta, w, w2, pr, m->desc.norm_eps, T, m->desc.d_model, out, m->stream);
  return launch_add_layernorm(x, delta, w, b, w2, b2, pr, m->desc.norm_eps, T, m->desc.d_model, out, m->stream);
}

// Up to three block linears that read the same input, in one launch.
static int linears(qzo_model* m, const Linear* const* Ls, __nv_bfloat16* const* outs, int n, int ldo,
                   const __nv_bfloat16* in, int T, uint64_t seed, int sign, float eps, int pair_rows) {
  GemmLinear g[kMaxGroupedLinears];
  double flops = 0.0;
  for (int j = 0; j < n; ++j) {
    g[j] = GemmLinear{Ls[j]->wq, m->scales + Ls[j]->idx_base, Ls[j]->bias, outs[j], ldo, Ls[j]->N,
                      (uint64_t)Ls[j]->idx_base};
    flops += 2.0 * T * (double)Ls[j]->K * (double)Ls[j]->N;
  }
  const bool timed = m->profiling && m->events_used + 2 <= m->events.size();
  if (timed) QZO_CUDA_TRY(cudaEventRecord(m->events[m->events_used], m->stream));
  QZO_TRY(launch_perturbed_gemm_group(in, T, Ls[0]->K, g, n, seed, sign, eps, pair_rows, m->gemm_ws, m->gemm_ws_bytes,
                                      m->status, m->stream, nullptr, m->cur_sp));
  if (timed) {
    QZO_CUDA_TRY(cudaEventRecord(m->events[m->events_used + 1], m->stream));
    m->events_used += 2;
    m->profiled_flops += flops;
  }
  return QZO_OK;
}
static int linear(qzo_model* m, const Linear& L, const __nv_bfloat16* in, __nv_bfloat16* out, int ldo, int T,
                  uint64_t seed, int sign, float eps, int pair_rows) {
  const Linear* Ls[1] = {&L};
  __nv_bfloat16* outs[1] = {out};
  return linears(m, Ls, outs, 1, ldo, in, T, seed, sign, eps, pair_rows);
}

// One forward pass and its loss.  paired: the batch is given twice (2 B sequences); the first copy
// is run with sign * eps, the second with -sign * eps, and d_loss[0], d_loss[1] receive the two mean
// losses.  Every kernel works row by row or sequence by sequence, so each half computes exactly what
// a pass of its own would.
// d_loss (mean, may be null) and d_sums (may be null) receive the result: single pass: d_loss[0], d_sums[0] = sum of
// token losses, d_sums[2] = kept tokens; paired: d_loss[0..1], d_sums[0..1] sums, d_sums[2..3] counts.
int forward_loss(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed, int sign,
                 float eps, float* d_loss, float* d_sums, bool paired, int slot = 0) {
  const qzo_model_desc& d = m->desc;
  const int dm = d.d_model, H = d.n_heads, dh = dm / H, F = d.d_ffn;
  const int pair_rows = paired ? B * S : 0;
  if (paired) B *= 2;
  const int T = B * S;
  cudaStream_t st = m->stream;
  const bool llama = d.arch == QZO_ARCH_LLAMA;
  const bool jp = m->joint && sign != 0;            // joint mode: the un-quantised tensors are perturbed too
  const int vpl = llama ? 2 : 4;                    // vectors per layer: norm1 gain (bias), norm2 gain (bias)
  if (jp) QZO_TRY(launch_perturb_vectors(m->vec_table, m->vec_base, m->n_vec, dm, seed, eps, m->vec_plus, m->vec_minus, st));
  QZO_TRY(launch_embedding(d_tokens, m->embed, llama ? nullptr : m->pos_embed, T, S, dm, d.vocab, m->x, m->status, seed,
                           (uint64_t)m->base_embed, jp ? (float)sign * eps : 0.0f, jp ? pair_rows : 0, st));
  // The residual stream x is updated lazily: a projection writes its output to xn, and the norm that
  // follows adds it to x before normalising (x += xn; xn = norm(x)).
  const __nv_bfloat16* pending = nullptr;          // projection output not yet added to x
  for (int li = 0; li < d.n_layers; ++li) {
    const Layer& L = m->layers[li];
    QZO_TRY(add_norm(m, m->x, pending, L.norm1_w, L.norm1_b, li * vpl, sign, pair_rows, T, m->xn));
    if (li > 0 && li - 1 == m->capture_layer)
      QZO_CUDA_TRY(cudaMemcpyAsync(m->capture, m->x, (size_t)T * dm * 2, cudaMemcpyDeviceToDevice, st));
    {
      const Linear* qkv_l[3] = {&L.lin[0], &L.lin[1], &L.lin[2]};
      __nv_bfloat16* qkv_o[3] = {m->qkv, m->qkv + dm, m->qkv + 2 * dm};
      QZO_TRY(linears(m, qkv_l, qkv_o, 3, 3 * dm, m->xn, T, seed, sign, eps, pair_rows));
    }
    if (llama) QZO_TRY(launch_rope(m->qkv, m->qkv + dm, 3 * dm, 3 * dm, m->rope_cs, T, S, H, dh, st));
    QZO_TRY(launch_attention(m->qkv, m->qkv + dm, m->qkv + 2 * dm, 3 * dm, 3 * dm, 3 * dm, m->att, dm, B, S, H, dh, st));
    QZO_TRY(linear(m, L.lin[3], m->att, m->xn, dm, T, seed, sign, eps, pair_rows));
    QZO_TRY(add_norm(m, m->x, m->xn, L.norm2_w, L.norm2_b, li * vpl + vpl / 2, sign, pair_rows, T, m->xn));
    if (llama) {
      const Linear* gu_l[2] = {&L.lin[4], &L.lin[5]};
      __nv_bfloat16* gu_o[2] = {m->mlp_a, m->mlp_b};
      QZO_TRY(linears(m, gu_l, gu_o, 2, F, m->xn, T, seed, sign, eps, pair_rows));
      QZO_TRY(launch_silu_mul(m->mlp_a, m->mlp_b, m->mlp_a, (int64_t)T * F, st));
      QZO_TRY(linear(m, L.lin[6], m->mlp_a, m->xn, dm, T, seed, sign, eps, pair_rows));
    } else {
      QZO_TRY(linear(m, L.lin[4], m->xn, m->mlp_a, F, T, seed, sign, eps, pair_rows));
      QZO_TRY(launch_relu(m->mlp_a, (int64_t)T * F, st));
      QZO_TRY(linear(m, L.lin[5], m->mlp_a, m->xn, dm, T, seed, sign, eps, pair_rows));
    }
    pending = m->xn;
  }
  QZO_TRY(add_norm(m, m->x, pending, m->final_norm_w, m->final_norm_b, d.n_layers * vpl, sign, pair_rows, T, m->xn));
  if (d.n_layers - 1 == m->capture_layer)
    QZO_CUDA_TRY(cudaMemcpyAsync(m->capture, m->x, (size_t)T * dm * 2, cudaMemcpyDeviceToDevice, st));
  if (jp) {
    // perturbed copies of the lm_head, rounded to its storage type; a paired pass needs both
    const int64_t cnt = (int64_t)d.vocab * dm;
    __nv_bfloat16* first = sign > 0 ? m->lm_plus : m->lm_minus;
    QZO_TRY(launch_perturb_dense_bf16(m->lm_head, first, cnt, seed, (uint64_t)m->base_lm_head, (float)sign * eps, st));
    if (paired) {
      __nv_bfloat16* second = sign > 0 ? m->lm_minus : m->lm_plus;
      QZO_TRY(launch_perturb_dense_bf16(m->lm_head, second, cnt, seed, (uint64_t)m->base_lm_head, -(float)sign * eps, st));
      QZO_TRY(launch_bf16_gemm_f32out(m->xn, first, m->logits, pair_rows, dm, d.vocab, m->status, st));
      QZO_TRY(launch_bf16_gemm_f32out(m->xn + (size_t)pair_rows * dm, second, m->logits + (size_t)pair_rows * d.vocab,
                                      T - pair_rows, dm, d.vocab, m->status, st));
    } else {
      QZO_TRY(launch_bf16_gemm_f32out(m->xn, first, m->logits, T, dm, d.vocab, m->status, st));
    }
  } else {
    QZO_TRY(launch_bf16_gemm_f32out(m->xn, m->lm_head, m->logits, T, dm, d.vocab, m->status, st));
  }
  if (paired) {
    const int Th = pair_rows;
    QZO_TRY(launch_cross_entropy(m->logits, d_labels, Th, d.vocab, m->row_loss, d_loss, d_sums, d_sums ? d_sums + 2 : nullptr, st));
    QZO_TRY(launch_cross_entropy(m->logits + (size_t)Th * d.vocab, d_labels + Th, Th, d.vocab, m->row_loss + Th,
                                 d_loss ? d_loss + 1 : nullptr, d_sums ? d_sums + 1 : nullptr, d_sums ? d_sums + 3 : nullptr, st));
  } else {
    QZO_TRY(launch_cross_entropy(m->logits, d_labels, T, d.vocab, m->row_loss, d_loss, d_sums ? d_sums + slot : nullptr,
                                 d_sums ? d_sums + 2 + slot : nullptr, st));
  }
  m->last_T = T;
  return QZO_OK;
}

int check_batch(const qzo_model* m, const void* tok, const void* lab, int B, int S) {
  if (!m || !tok || !lab || B <= 0 || S <= 0) return QZO_ERR_BAD_ARG;
  if (S > m->desc.max_seq) return QZO_ERR_BAD_ARG;
  if ((int64_t)B * S > m->max_tokens) return QZO_ERR_WORKSPACE;
  return QZO_OK;
}

int update_all_scales(qzo_model* m, uint64_t seed, float coef_host, const float* coef_dev) {
  return launch_update_scales(m->scales, m->flat_entries, seed, 0, coef_host, coef_dev, m->stream);
}

// First half of a step: both perturbed forwards (Algorithm 1, the two forward passes on the same batch and
// seed); d_sums receives {sum of token losses (+), the same (-), kept tokens (+), kept tokens (-)}.
int step_begin(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed, float eps,
               float* d_sums) {
  const int T = B * S;
  if (paired_rows_ok(2 * T, T)) {
    // both passes as one forward over two copies of the batch (the workspace holds 2 * max_tokens rows)
    const size_t bytes = (size_t)T * sizeof(int32_t);
    if (d_tokens != m->tok_dev)
      QZO_CUDA_TRY(cudaMemcpyAsync(m->tok_dev, d_tokens, bytes, cudaMemcpyDeviceToDevice, m->stream));
    if (d_labels != m->lab_dev)
      QZO_CUDA_TRY(cudaMemcpyAsync(m->lab_dev, d_labels, bytes, cudaMemcpyDeviceToDevice, m->stream));
    QZO_CUDA_TRY(cudaMemcpyAsync(m->tok_dev + T, m->tok_dev, bytes, cudaMemcpyDeviceToDevice, m->stream));
    QZO_CUDA_TRY(cudaMemcpyAsync(m->lab_dev + T, m->lab_dev, bytes, cudaMemcpyDeviceToDevice, m->stream));
    QZO_TRY(forward_loss(m, m->tok_dev, m->lab_dev, B, S, seed, +1, eps, m->loss2, d_sums, true));
  } else {
    QZO_TRY(forward_loss(m, d_tokens, d_labels, B, S, seed, +1, eps, m->loss2, d_sums, false, 0));
    QZO_TRY(forward_loss(m, d_tokens, d_labels, B, S, seed, -1, eps, m->loss2 + 1, d_sums, false, 1));
  }
  return QZO_OK;
}

// Second half: d, d' (Eq. 6) and the seeded update from the loss sums, all on the device.  With h_out the
// stream is synchronised and what the device found is reported; the scales are untouched in every error case.
static int step_finish_launches(qzo_model* m, const float* d_sums, uint64_t seed, float eps, float lr, float clip) {
  QZO_TRY(launch_ddc(d_sums, eps, lr, m->joint ? m->lr_dense : 0.0f, clip, m->status, m->out7, m->stream));
  QZO_TRY(update_all_scales(m, seed, 0.0f, m->out7 + 4));
  if (m->joint) {
    // ZO-SGD on the un-quantised tensors with the same clipped d' and the same z stream (Def. 3.2)
    const int64_t cnt = (int64_t)m->desc.vocab * m->desc.d_model;
    const float* coef = m->out7 + 6;
    QZO_TRY(launch_update_dense_bf16(const_cast<__nv_bfloat16*>(m->embed), cnt, seed, (uint64_t)m->base_embed, coef, m->stream));
    QZO_TRY(launch_update_dense_bf16(const_cast<__nv_bfloat16*>(m->lm_head), cnt, seed, (uint64_t)m->base_lm_head, coef, m->stream));
    QZO_TRY(launch_update_vectors(const_cast<float* const*>(reinterpret_cast<const float* const*>(m->vec_table)), m->vec_base,
                                  m->n_vec, m->desc.d_model, seed, coef, m->stream));
  }
  return QZO_OK;
}

// What the device found in the step just launched (synchronises the stream): l+, l-, d, d' and the error, if any.
static int read_step_result(qzo_model* m, float* h_out) {
  {
    float host[6];
    QZO_CUDA_TRY(cudaMemcpyAsync(host, m->out7, sizeof(host), cudaMemcpyDeviceToHost, m->stream));
    QZO_CUDA_TRY(cudaStreamSynchronize(m->stream));
    memcpy(h_out, host, 4 * sizeof(float));
    const int st = (int)host[5];
    if (st & kStatusTimeout) return QZO_ERR_DEVICE_TIMEOUT;
    if (st & kStatusBadToken) return QZO_ERR_BAD_ARG;
    if (!std::isfinite(host[0]) || !std::isfinite(host[1])) return QZO_ERR_NONFINITE;
  }
  return QZO_OK;
}

int step_finish(qzo_model* m, const float* d_sums, uint64_t seed, float eps, float lr, float clip, float* h_out) {
  QZO_TRY(step_finish_launches(m, d_sums, seed, eps, lr, clip));
  return h_out ? read_step_result(m, h_out) : QZO_OK;
}

constexpr size_t kMaxRecordedShapes = 16;

// Records the launch sequence of a step's two forwards on (B, S) into a CUDA graph.  Their GEMMs take seed and eps
// from m->sp_dev, the tokens come from the model's own buffers and the loss sums go to m->sums, so the graph serves
// every later step of that shape.  Nothing runs while recording.  A failure ends the recording and switches
// recorded steps off.
static int record_forwards(qzo_model* m, int B, int S, qzo_model::RecordedStep* rec) {
  const long long before = launch_count();
  // recorded on a stream of the model's own (the caller's may be the legacy default stream, which cannot
  // record); the graph is then launched on the caller's stream
  if (m->rec_stream == nullptr && cudaStreamCreateWithFlags(&m->rec_stream, cudaStreamNonBlocking) != cudaSuccess) {
    (void)cudaGetLastError();
    m->rec_stream = nullptr;
    return QZO_ERR_CUDA;
  }
  if (cudaStreamBeginCapture(m->rec_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    (void)cudaGetLastError();
    return QZO_ERR_CUDA;
  }
  cudaStream_t const callers = m->stream;
  m->stream = m->rec_stream;
  m->cur_sp = m->sp_dev;
  int rc = step_begin(m, m->tok_dev, m->lab_dev, B, S, 0, 1.0f, m->sums);
  m->cur_sp = nullptr;
  m->stream = callers;
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(m->rec_stream, &graph);
  if (rc == QZO_OK && (e != cudaSuccess || graph == nullptr)) rc = QZO_ERR_CUDA;
  if (rc == QZO_OK && cudaGraphInstantiate(&rec->exec, graph, 0) != cudaSuccess) rc = QZO_ERR_CUDA;
  if (graph) cudaGraphDestroy(graph);
  rec->launches = launch_count() - before;
  rec->rows = m->last_T;
  add_launches(-rec->launches);             // recorded, not run: a replay counts them
  if (rc != QZO_OK) {
    (void)cudaGetLastError();
    rec->exec = nullptr;
    return rc;
  }
  return QZO_OK;
}

// The two forwards of a step (step_begin), replayed from a recording where there is one.  A launch sequence that
// depends on nothing but (B, S) is recorded once and replayed: with few tokens the host would otherwise need longer
// to issue the launches than the device needs to run them.
int step_begin_replayed(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed,
                        float eps, float* d_sums) {
  const long long shape = ((long long)B << 32) | (long long)S;
  // at most kMaxRecordedShapes batch shapes are recorded per model; further shapes run the direct way
  const bool replay = m->use_graphs && !m->joint && m->capture_layer < 0 && !m->profiling &&
                      (m->recorded.size() < kMaxRecordedShapes || m->recorded.count(shape) > 0);
  if (replay) {
    qzo_model::RecordedStep& rec = m->recorded[shape];
    if (rec.seen) {
      const size_t bytes = (size_t)B * S * sizeof(int32_t);
      if (d_tokens != m->tok_dev)
        QZO_CUDA_TRY(cudaMemcpyAsync(m->tok_dev, d_tokens, bytes, cudaMemcpyDeviceToDevice, m->stream));
      if (d_labels != m->lab_dev)
        QZO_CUDA_TRY(cudaMemcpyAsync(m->lab_dev, d_labels, bytes, cudaMemcpyDeviceToDevice, m->stream));
      if (rec.exec == nullptr && record_forwards(m, B, S, &rec) != QZO_OK) m->use_graphs = false;
      if (rec.exec != nullptr) {
        QZO_TRY(launch_set_step_params(m->sp_dev, seed, eps, m->stream));
        QZO_CUDA_TRY(cudaGraphLaunch(rec.exec, m->stream));
        add_launches(rec.launches);
        m->last_T = rec.rows;
        if (d_sums != m->sums)
          QZO_CUDA_TRY(cudaMemcpyAsync(d_sums, m->sums, 4 * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
        return QZO_OK;
      }
      d_tokens = m->tok_dev;
      d_labels = m->lab_dev;
    }
    rec.seen = true;                          // the first step of a shape runs the direct way
  }
  return step_begin(m, d_tokens, d_labels, B, S, seed, eps, d_sums);
}

int step_device(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed, float eps,
                float lr, float clip, float* h_out) {
  QZO_TRY(step_begin_replayed(m, d_tokens, d_labels, B, S, seed, eps, m->sums));
  return step_finish(m, m->sums, seed, eps, lr, clip, h_out);
}

// (layer, linear) of a flat linear id, or false when it is out of range.
bool split_linear_id(const qzo_model* m, int linear_id, int* layer, int* linear) {
  if (linear_id < 0 || linear_id >= m->desc.n_layers * m->n_lin) return false;
  *layer = linear_id / m->n_lin;
  *linear = linear_id % m->n_lin;
  return true;
}

}  // namespace qzo

// =========================================================================================
// C ABI
// =========================================================================================
using namespace qzo;

extern "C" {

const char* qzo_strerror(int status) {
  switch (status) {
    case QZO_OK: return "ok";
    case QZO_ERR_BAD_ARG: return "bad argument";
    case QZO_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs compute capability 10.x; no other backend)";
    case QZO_ERR_WORKSPACE: return "workspace too small or misaligned";
    case QZO_ERR_NONFINITE: return "non-finite loss or directional derivative; scales untouched";
    case QZO_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case QZO_ERR_CUDA: return "CUDA call failed (see qzo_last_cuda_error)";
    case QZO_ERR_MISSING_TENSOR: return "a required tensor was not supplied";
    default: return "unknown status";
  }
}

int qzo_last_cuda_error(void) { return qzo::last_cuda_error(); }
int64_t qzo_launch_count(void) { return (int64_t)qzo::launch_count(); }

int qzo_philox_words(uint64_t seed, uint64_t block_base, int64_t n_blocks, uint32_t* d_words, float* d_uniforms,
                     void* stream) {
  if (n_blocks < 0 || (n_blocks > 0 && !d_words)) return QZO_ERR_BAD_ARG;
  QZO_TRY(check_device());
  return launch_philox_words(seed, block_base, n_blocks, d_words, d_uniforms, (cudaStream_t)stream);
}

int qzo_normals(uint64_t seed, uint64_t index_base, int64_t count, float* d_z, void* stream) {
  if (count < 0 || (count > 0 && !d_z)) return QZO_ERR_BAD_ARG;
  QZO_TRY(check_device());
  return launch_normals(seed, index_base, count, d_z, (cudaStream_t)stream);
}

int qzo_quantize_int4(const float* d_w, int K, int N, uint32_t* d_qpacked, void* d_scales_bf16, void* stream) {
  if (!d_w || !d_qpacked || !d_scales_bf16 || K <= 0 || N <= 0 || (K % 8)) return QZO_ERR_BAD_ARG;
  QZO_TRY(check_device());
  return launch_quantize(d_w, K, N, d_qpacked, (__nv_bfloat16*)d_scales_bf16, (cudaStream_t)stream);
}

int qzo_unpack_int4(const uint32_t* d_qpacked, int K, int N, int8_t* d_q, void* stream) {
  if (!d_qpacked || !d_q || K <= 0 || N <= 0 || (K % 8)) return QZO_ERR_BAD_ARG;
  QZO_TRY(check_device());
  return launch_unpack(d_qpacked, K, N, d_q, (cudaStream_t)stream);
}

int qzo_repacked_bytes(int K, int N, size_t* bytes) {
  if (!bytes || K <= 0 || N <= 0 || (K % 8)) return QZO_ERR_BAD_ARG;
  *bytes = repacked_bytes(K, N);
  return QZO_OK;
}

int qzo_repack_int4(const uint32_t* d_qpacked, int K, int N, void* d_out, size_t out_bytes, void* stream) {
  if (!d_qpacked || !d_out || K <= 0 || N <= 0 || (K % 8)) return QZO_ERR_BAD_ARG;
  if (out_bytes < repacked_bytes(K, N) || ((uintptr_t)d_out & 255)) return QZO_ERR_WORKSPACE;
  QZO_TRY(check_device());
  return launch_repack(d_qpacked, K, N, d_out, (cudaStream_t)stream);
}

int qzo_unpack_kernel_layout(const void* d_wq, int K, int N, int8_t* d_q, void* stream) {
  if (!d_wq || !d_q || K <= 0 || N <= 0 || (K % 8)) return QZO_ERR_BAD_ARG;
  QZO_TRY(check_device());
  return launch_unpack_kernel_layout(d_wq, K, N, d_q, (cudaStream_t)stream);
}

int qzo_gemm_workspace_bytes(int M, int K, int N, size_t* bytes) {
  if (!bytes || M <= 0 || K <= 0 || N <= 0) return QZO_ERR_BAD_ARG;
  *bytes = gemm_workspace_bytes(M, K, N);
  return QZO_OK;
}

int qzo_perturbed_gemm(const void* d_x_bf16, const void* d_wq, const void* d_scales_bf16, const float* d_bias,
                       void* d_y_bf16, int M, int K, int N, uint64_t seed, uint64_t scale_index_base, int sign,
                       float eps, void* d_workspace, size_t workspace_bytes, int* d_status, void* stream) {
  if (!d_x_bf16 || !d_wq || !d_scales_bf16 || !d_y_bf16) return QZO_ERR_BAD_ARG;
  if (sign < -1 || sign > 1 || !(eps > 0.0f)) return QZO_ERR_BAD_ARG;
  if (((uintptr_t)d_x_bf16 & 15) || ((uintptr_t)d_wq & 15) || ((uintptr_t)d_scales_bf16 & 15) ||
      ((uintptr_t)d_y_bf16 & 15))
    return QZO_ERR_BAD_ARG;
  if (d_workspace && ((uintptr_t)d_workspace & 255)) return QZO_ERR_WORKSPACE;
  QZO_TRY(check_device());
  if (N <= 0 || (N % 8)) return QZO_ERR_BAD_ARG;
  const GemmLinear g{d_wq, (const __nv_bfloat16*)d_scales_bf16, d_bias, (__nv_bfloat16*)d_y_bf16, N, N,
                     scale_index_base};
  return launch_perturbed_gemm_group((const __nv_bfloat16*)d_x_bf16, M, K, &g, 1, seed, sign, eps, 0, d_workspace,
                                     workspace_bytes, d_status, (cudaStream_t)stream);
}

int qzo_perturbed_gemm_table16(const void* d_x_bf16, const void* d_codes, const void* d_scales_bf16, const float* h_table16,
                               const float* d_bias, void* d_y_bf16, int M, int K, int N, uint64_t seed,
                               uint64_t scale_index_base, int sign, float eps, void* d_workspace, size_t workspace_bytes,
                               int* d_status, void* stream) {
  if (!d_x_bf16 || !d_codes || !d_scales_bf16 || !d_y_bf16 || !h_table16) return QZO_ERR_BAD_ARG;
  if (sign < -1 || sign > 1 || !(eps > 0.0f)) return QZO_ERR_BAD_ARG;
  for (int i = 0; i < 16; ++i)
    if (!std::isfinite(h_table16[i])) return QZO_ERR_BAD_ARG;
  if (((uintptr_t)d_x_bf16 & 15) || ((uintptr_t)d_codes & 15) || ((uintptr_t)d_scales_bf16 & 15) ||
      ((uintptr_t)d_y_bf16 & 15))
    return QZO_ERR_BAD_ARG;
  if (d_workspace && ((uintptr_t)d_workspace & 255)) return QZO_ERR_WORKSPACE;
  QZO_TRY(check_device());
  if (N <= 0 || (N % 8)) return QZO_ERR_BAD_ARG;
  const GemmLinear g{d_codes, (const __nv_bfloat16*)d_scales_bf16, d_bias, (__nv_bfloat16*)d_y_bf16, N, N,
                     scale_index_base};
  return launch_perturbed_gemm_group((const __nv_bfloat16*)d_x_bf16, M, K, &g, 1, seed, sign, eps, 0, d_workspace,
                                     workspace_bytes, d_status, (cudaStream_t)stream, h_table16);
}

int qzo_perturbed_gemm_codebook16_channelwise(const void* d_x_bf16, const void* d_codes, const void* d_scales_bf16,
                                              const float* h_table16, const float* d_bias, void* d_y_bf16, int M, int K, int N,
                                              uint64_t seed, uint64_t scale_index_base, int sign, float eps,
                                              void* d_workspace, size_t workspace_bytes, int* d_status, void* stream) {
  if (!d_x_bf16 || !d_codes || !d_scales_bf16 || !d_y_bf16 || !h_table16) return QZO_ERR_BAD_ARG;
  if (sign < -1 || sign > 1 || !(eps > 0.0f)) return QZO_ERR_BAD_ARG;
  for (int i = 0; i < 16; ++i)
    if (!std::isfinite(h_table16[i])) return QZO_ERR_BAD_ARG;
  if (((uintptr_t)d_x_bf16 & 15) || ((uintptr_t)d_codes & 15) || ((uintptr_t)d_scales_bf16 & 15) ||
      ((uintptr_t)d_y_bf16 & 15))
    return QZO_ERR_BAD_ARG;
  if (d_workspace && ((uintptr_t)d_workspace & 255)) return QZO_ERR_WORKSPACE;
  QZO_TRY(check_device());
  if (N <= 0 || (N % 8)) return QZO_ERR_BAD_ARG;
  const GemmLinear g{d_codes, (const __nv_bfloat16*)d_scales_bf16, d_bias, (__nv_bfloat16*)d_y_bf16, N, N,
                     scale_index_base};
  return launch_perturbed_gemm_group((const __nv_bfloat16*)d_x_bf16, M, K, &g, 1, seed, sign, eps, 0, d_workspace,
                                     workspace_bytes, d_status, (cudaStream_t)stream, h_table16, nullptr, true);
}

int qzo_debug_gemm_wait_expiry(const void* d_x_bf16, const void* d_wq, const void* d_scales_bf16, void* d_y_bf16, int M,
                               int K, int N, int skip_group, int64_t wait_limit_cycles, int* d_status, void* stream) {
  if (skip_group < 0 || wait_limit_cycles <= 0 || !d_status) return QZO_ERR_BAD_ARG;
  set_gemm_wait_debug((long long)wait_limit_cycles, skip_group);
  const int rc = qzo_perturbed_gemm(d_x_bf16, d_wq, d_scales_bf16, nullptr, d_y_bf16, M, K, N, 1, 0, +1, 1e-3f, nullptr, 0,
                                    d_status, stream);
  set_gemm_wait_debug(0, -1);
  return rc;
}

int qzo_update_scales_flat(void* d_scales_bf16, int64_t count, uint64_t seed, uint64_t index_base, float lr, float g,
                           float clip, void* stream) {
  if (!d_scales_bf16 || count < 0 || (index_base % 4) || ((uintptr_t)d_scales_bf16 & 7) || !(clip >= 0.0f))
    return QZO_ERR_BAD_ARG;
  if (!std::isfinite(g) || !std::isfinite(lr)) return QZO_ERR_NONFINITE;
  QZO_TRY(check_device());
  const float gc = fminf(fmaxf(g, -clip), clip);
  const float coef = lr * gc;
  return launch_update_scales((__nv_bfloat16*)d_scales_bf16, count, seed, index_base, coef, nullptr, (cudaStream_t)stream);
}

int qzo_num_scales(const qzo_model_desc* desc, int64_t* flat_entries, int64_t* trainable) {
  QZO_TRY(validate_desc(desc));
  int64_t train = 0;
  const int64_t flat = scale_layout(*desc, -1, -1, nullptr, nullptr, &train);
  if (flat_entries) *flat_entries = flat;
  if (trainable) *trainable = train;
  return QZO_OK;
}

int qzo_scale_layout(const qzo_model_desc* desc, int layer, int linear, int64_t* index_base, int* G, int* N) {
  QZO_TRY(validate_desc(desc));
  LinearShape ls[7];
  const int nl = linear_shapes(*desc, ls);
  if (layer < 0 || layer >= desc->n_layers || linear < 0 || linear >= nl) return QZO_ERR_BAD_ARG;
  const int64_t b = scale_layout(*desc, layer, linear, G, N, nullptr);
  if (index_base) *index_base = b;
  return QZO_OK;
}

int qzo_workspace_bytes(const qzo_model_desc* desc, int max_tokens, size_t* bytes) {
  QZO_TRY(validate_desc(desc));
  if (!bytes || max_tokens <= 0) return QZO_ERR_BAD_ARG;
  WsPlan p;
  QZO_TRY(plan_workspace(*desc, max_tokens, &p));
  *bytes = p.total;
  return QZO_OK;
}

int qzo_init_model(const qzo_model_desc* desc, const qzo_tensor* tensors, int n_tensors, void* d_workspace,
                   size_t workspace_bytes, int max_tokens, void* stream, qzo_model** out) {
  QZO_TRY(validate_desc(desc));
  if (!tensors || n_tensors <= 0 || !out || max_tokens <= 0) return QZO_ERR_BAD_ARG;
  if (!d_workspace || ((uintptr_t)d_workspace & 255)) return QZO_ERR_WORKSPACE;
  QZO_TRY(check_device());
  WsPlan p;
  QZO_TRY(plan_workspace(*desc, max_tokens, &p));
  if (workspace_bytes < p.total) return QZO_ERR_WORKSPACE;

  std::map<std::string, const qzo_tensor*> by_name;
  for (int i = 0; i < n_tensors; ++i)
    if (tensors[i].name && tensors[i].dptr) by_name[tensors[i].name] = &tensors[i];
  int err = QZO_OK;
  auto get = [&](const std::string& name, int dtype, int64_t rows, int64_t cols) -> void* {
    auto it = by_name.find(name);
    if (it == by_name.end()) { if (err == QZO_OK) err = QZO_ERR_MISSING_TENSOR; return nullptr; }
    const qzo_tensor* t = it->second;
    if (t->dtype != dtype || t->shape[0] != rows || t->shape[1] != cols || ((uintptr_t)t->dptr & 15)) {
      if (err == QZO_OK) err = QZO_ERR_BAD_ARG;
      return nullptr;
    }
    return t->dptr;
  };

  qzo_model* m = new qzo_model();
  m->desc = *desc;
  m->stream = (cudaStream_t)stream;
  m->max_tokens = max_tokens;
  const bool opt = desc->arch == QZO_ARCH_OPT;
  const int dm = desc->d_model;
  int64_t train = 0;
  m->flat_entries = scale_layout(*desc, -1, -1, nullptr, nullptr, &train);
  m->embed = (const __nv_bfloat16*)get("embed", QZO_DTYPE_BF16, desc->vocab, dm);
  m->lm_head = (const __nv_bfloat16*)get("lm_head", QZO_DTYPE_BF16, desc->vocab, dm);
  if (opt) m->pos_embed = (const __nv_bfloat16*)get("pos_embed", QZO_DTYPE_BF16, desc->max_seq, dm);
  m->final_norm_w = (const float*)get("final_norm_w", QZO_DTYPE_F32, dm, 1);
  if (opt) m->final_norm_b = (const float*)get("final_norm_b", QZO_DTYPE_F32, dm, 1);
  m->scales = (__nv_bfloat16*)get("scales", QZO_DTYPE_BF16, m->flat_entries, 1);

  uint8_t* ws = (uint8_t*)d_workspace;
  LinearShape ls[7];
  m->n_lin = linear_shapes(*desc, ls);
  m->layers.resize(desc->n_layers);
  size_t woff = p.off_weights;
  for (int li = 0; li < desc->n_layers && err == QZO_OK; ++li) {
    Layer& L = m->layers[li];
    const std::string pre = "L" + std::to_string(li) + ".";
    L.norm1_w = (const float*)get(pre + "norm1_w", QZO_DTYPE_F32, dm, 1);
    L.norm2_w = (const float*)get(pre + "norm2_w", QZO_DTYPE_F32, dm, 1);
    if (opt) {
      L.norm1_b = (const float*)get(pre + "norm1_b", QZO_DTYPE_F32, dm, 1);
      L.norm2_b = (const float*)get(pre + "norm2_b", QZO_DTYPE_F32, dm, 1);
    }
    for (int i = 0; i < m->n_lin; ++i) {
      Linear& lin = L.lin[i];
      lin.K = ls[i].K; lin.N = ls[i].N;
      lin.idx_base = scale_layout(*desc, li, i, nullptr, nullptr, nullptr);
      const uint32_t* qw = (const uint32_t*)get(pre + ls[i].name + ".qweight", QZO_DTYPE_U32, lin.K / 8, lin.N);
      if (opt) lin.bias = (const float*)get(pre + ls[i].name + ".bias", QZO_DTYPE_F32, lin.N, 1);
      if (err != QZO_OK) break;
      lin.wq = ws + woff;
      int s = launch_repack(qw, lin.K, lin.N, ws + woff, m->stream);
      if (s != QZO_OK) { err = s; break; }
      woff += align_up(repacked_bytes(lin.K, lin.N), 256);
    }
  }
  if (err != QZO_OK) { delete m; return err; }

  m->x = (__nv_bfloat16*)(ws + p.off_x);
  m->xn = (__nv_bfloat16*)(ws + p.off_xn);
  m->qkv = (__nv_bfloat16*)(ws + p.off_qkv);
  m->att = (__nv_bfloat16*)(ws + p.off_att);
  m->mlp_a = (__nv_bfloat16*)(ws + p.off_a);
  m->mlp_b = (__nv_bfloat16*)(ws + p.off_b);
  m->capture = (__nv_bfloat16*)(ws + p.off_capture);
  m->logits = (float*)(ws + p.off_logits);
  m->row_loss = (float*)(ws + p.off_rowloss);
  float* scal = (float*)(ws + p.off_scalars);
  m->loss2 = scal;            // [0], [1]
  m->sums = scal + 4;         // [4..7]
  m->out7 = scal + 8;         // [8..14]
  m->status = (int*)(scal + 32);
  m->sp_dev = reinterpret_cast<StepParams*>(scal + 40);
  m->rope_cs = (float*)(ws + p.off_rope);
  m->tok_dev = (int32_t*)(ws + p.off_tok);
  m->lab_dev = (int32_t*)(ws + p.off_lab);
  m->gemm_ws = ws + p.off_gemm;
  m->gemm_ws_bytes = p.gemm_bytes;
  cudaError_t ce = cudaMemsetAsync(scal, 0, 64 * 4, m->stream);
  if (ce != cudaSuccess) { set_last_cuda_error(ce); delete m; return QZO_ERR_CUDA; }
  if (!opt) {
    int s = launch_rope_table(m->rope_cs, desc->max_seq, dm / desc->n_heads, desc->rope_theta, m->stream);
    if (s != QZO_OK) { delete m; return s; }
  }
  *out = m;
  return QZO_OK;
}

int qzo_profile_gemms(qzo_model* m, int max_launches) {
  if (!m || max_launches < 0) return QZO_ERR_BAD_ARG;
  for (cudaEvent_t e : m->events) cudaEventDestroy(e);
  m->events.clear();
  m->events_used = 0;
  m->profiled_flops = 0.0;
  m->profiling = max_launches > 0;
  for (int i = 0; i < 2 * max_launches; ++i) {
    cudaEvent_t e;
    QZO_CUDA_TRY(cudaEventCreate(&e));
    m->events.push_back(e);
  }
  return QZO_OK;
}

int qzo_profile_read(qzo_model* m, int64_t* launches, double* total_ms, double* total_flops) {
  if (!m || !launches || !total_ms || !total_flops) return QZO_ERR_BAD_ARG;
  QZO_CUDA_TRY(cudaStreamSynchronize(m->stream));
  double ms = 0.0;
  for (size_t i = 0; i + 1 < m->events_used; i += 2) {
    float t = 0.0f;
    QZO_CUDA_TRY(cudaEventElapsedTime(&t, m->events[i], m->events[i + 1]));
    ms += t;
  }
  *launches = (int64_t)(m->events_used / 2);
  *total_ms = ms;
  *total_flops = m->profiled_flops;
  m->events_used = 0;
  m->profiled_flops = 0.0;
  return QZO_OK;
}

int qzo_free_model(qzo_model* m) {
  if (!m) return QZO_ERR_BAD_ARG;
  for (cudaEvent_t e : m->events) cudaEventDestroy(e);
  for (auto& kv : m->recorded)
    if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
  if (m->rec_stream) cudaStreamDestroy(m->rec_stream);
  delete m;
  return QZO_OK;
}

int qzo_forward_loss(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed,
                     int sign, float eps, float* d_loss) {
  QZO_TRY(check_batch(m, d_tokens, d_labels, B, S));
  if (!d_loss || sign < -1 || sign > 1 || !(eps > 0.0f)) return QZO_ERR_BAD_ARG;
  return forward_loss(m, d_tokens, d_labels, B, S, seed, sign, eps, d_loss, nullptr, false);
}

int qzo_update_scales(qzo_model* m, uint64_t seed, float lr, float g, float clip) {
  if (!m || !(clip >= 0.0f)) return QZO_ERR_BAD_ARG;
  if (!std::isfinite(g) || !std::isfinite(lr)) return QZO_ERR_NONFINITE;
  const float gc = fminf(fmaxf(g, -clip), clip);
  return update_all_scales(m, seed, lr * gc, nullptr);
}

int qzo_step(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed, float eps,
             float lr, float clip, float* h_out) {
  QZO_TRY(check_batch(m, d_tokens, d_labels, B, S));
  if (!(eps > 0.0f) || !(clip >= 0.0f) || !std::isfinite(lr)) return QZO_ERR_BAD_ARG;
  return step_device(m, d_tokens, d_labels, B, S, seed, eps, lr, clip, h_out);
}

int qzo_use_recorded_steps(qzo_model* m, int on) {
  if (!m) return QZO_ERR_BAD_ARG;
  m->use_graphs = on != 0;
  return QZO_OK;
}

int qzo_recorded_step_count(qzo_model* m, int* h_count) {
  if (!m || !h_count) return QZO_ERR_BAD_ARG;
  int n = 0;
  for (const auto& kv : m->recorded) n += kv.second.exec != nullptr;
  *h_count = m->use_graphs ? n : -1;
  return QZO_OK;
}

int qzo_step_host(qzo_model* m, const int32_t* h_tokens, const int32_t* h_labels, int B, int S, uint64_t seed,
                  float eps, float lr, float clip, float* h_out) {
  QZO_TRY(check_batch(m, h_tokens, h_labels, B, S));
  if (!(eps > 0.0f) || !(clip >= 0.0f) || !std::isfinite(lr) || !h_out) return QZO_ERR_BAD_ARG;
  const size_t bytes = (size_t)B * S * sizeof(int32_t);
  QZO_CUDA_TRY(cudaMemcpyAsync(m->tok_dev, h_tokens, bytes, cudaMemcpyHostToDevice, m->stream));
  QZO_CUDA_TRY(cudaMemcpyAsync(m->lab_dev, h_labels, bytes, cudaMemcpyHostToDevice, m->stream));
  return step_device(m, m->tok_dev, m->lab_dev, B, S, seed, eps, lr, clip, h_out);
}

int qzo_step_begin(qzo_model* m, const int32_t* d_tokens, const int32_t* d_labels, int B, int S, uint64_t seed,
                   float eps, float* d_sums) {
  QZO_TRY(check_batch(m, d_tokens, d_labels, B, S));
  if (!(eps > 0.0f) || !d_sums || ((uintptr_t)d_sums & 15)) return QZO_ERR_BAD_ARG;
  return step_begin_replayed(m, d_tokens, d_labels, B, S, seed, eps, d_sums);
}

int qzo_step_finish(qzo_model* m, const float* d_sums, uint64_t seed, float eps, float lr, float clip, float* h_out) {
  if (!m || !d_sums || ((uintptr_t)d_sums & 15)) return QZO_ERR_BAD_ARG;
  if (!(eps > 0.0f) || !(clip >= 0.0f) || !std::isfinite(lr)) return QZO_ERR_BAD_ARG;
  return step_finish(m, d_sums, seed, eps, lr, clip, h_out);
}

static size_t joint_bytes(const qzo_model_desc& d, int* n_vec_out) {
  const int n_vec = (2 * d.n_layers + 1) * (d.arch == QZO_ARCH_OPT ? 2 : 1);
  if (n_vec_out) *n_vec_out = n_vec;
  size_t off = 0;
  auto take = [&](size_t bytes) { off = (off + bytes + 255) / 256 * 256; };
  take((size_t)n_vec * 8);                         // pointer table
  take((size_t)n_vec * 8);                         // index bases
  take((size_t)n_vec * d.d_model * 4);             // vectors, +eps
  take((size_t)n_vec * d.d_model * 4);             // vectors, -eps
  take((size_t)d.vocab * d.d_model * 2);           // lm_head, +eps
  take((size_t)d.vocab * d.d_model * 2);           // lm_head, -eps
  return off;
}

int qzo_joint_workspace_bytes(const qzo_model_desc* desc, size_t* bytes) {
  QZO_TRY(validate_desc(desc));
  if (!bytes) return QZO_ERR_BAD_ARG;
  *bytes = joint_bytes(*desc, nullptr);
  return QZO_OK;
}

int qzo_enable_joint_spsa(qzo_model* m, void* d_workspace, size_t workspace_bytes, float lr_dense) {
  if (!m) return QZO_ERR_BAD_ARG;
  if (!d_workspace) { m->joint = false; return QZO_OK; }
  if (!std::isfinite(lr_dense)) return QZO_ERR_BAD_ARG;
  if ((uintptr_t)d_workspace & 255) return QZO_ERR_WORKSPACE;
  const qzo_model_desc& d = m->desc;
  int n_vec = 0;
  if (workspace_bytes < joint_bytes(d, &n_vec)) return QZO_ERR_WORKSPACE;
  const bool opt = d.arch == QZO_ARCH_OPT;
  // index ranges: after the scales, each base rounded up to a multiple of 8: embedding, lm_head, then the
  // norm vectors layer by layer (gain, bias), the final norm last
  int64_t run = m->flat_entries;
  auto next_base = [&](int64_t count) { run = (run + 7) / 8 * 8; const int64_t b = run; run += count; return b; };
  m->base_embed = next_base((int64_t)d.vocab * d.d_model);
  m->base_lm_head = next_base((int64_t)d.vocab * d.d_model);
  std::vector<const float*> ptrs;
  std::vector<unsigned long long> bases;
  auto add_vec = [&](const float* p) { ptrs.push_back(p); bases.push_back((unsigned long long)next_base(d.d_model)); };
  for (int li = 0; li < d.n_layers; ++li) {
    const Layer& L = m->layers[li];
    add_vec(L.norm1_w); if (opt) add_vec(L.norm1_b);
    add_vec(L.norm2_w); if (opt) add_vec(L.norm2_b);
  }
  add_vec(m->final_norm_w); if (opt) add_vec(m->final_norm_b);
  uint8_t* ws = (uint8_t*)d_workspace;
  size_t off = 0;
  auto take = [&](size_t bytes) { uint8_t* p = ws + off; off = (off + bytes + 255) / 256 * 256; return p; };
  const float** tab = (const float**)take((size_t)n_vec * 8);
  unsigned long long* bas = (unsigned long long*)take((size_t)n_vec * 8);
  m->vec_plus = (float*)take((size_t)n_vec * d.d_model * 4);
  m->vec_minus = (float*)take((size_t)n_vec * d.d_model * 4);
  m->lm_plus = (__nv_bfloat16*)take((size_t)d.vocab * d.d_model * 2);
  m->lm_minus = (__nv_bfloat16*)take((size_t)d.vocab * d.d_model * 2);
  QZO_CUDA_TRY(cudaMemcpyAsync(tab, ptrs.data(), (size_t)n_vec * 8, cudaMemcpyHostToDevice, m->stream));
  QZO_CUDA_TRY(cudaMemcpyAsync(bas, bases.data(), (size_t)n_vec * 8, cudaMemcpyHostToDevice, m->stream));
  QZO_CUDA_TRY(cudaStreamSynchronize(m->stream));      // the host vectors go out of scope
  m->vec_table = tab;
  m->vec_base = bas;
  m->n_vec = n_vec;
  m->lr_dense = lr_dense;
  m->joint = true;
  return QZO_OK;
}

int qzo_get_scales(qzo_model* m, int linear_id, void* d_bf16, size_t bytes) {
  if (!m || !d_bf16) return QZO_ERR_BAD_ARG;
  const __nv_bfloat16* src = m->scales;
  size_t need = (size_t)m->flat_entries * 2;
  if (linear_id != -1) {
    int layer = 0, linear = 0;
    if (!split_linear_id(m, linear_id, &layer, &linear)) return QZO_ERR_BAD_ARG;
    const Linear& L = m->layers[layer].lin[linear];
    src = m->scales + L.idx_base;
    need = (size_t)ceil_div(L.K, kGroup) * L.N * 2;
  }
  if (bytes != need) return QZO_ERR_BAD_ARG;
  QZO_CUDA_TRY(cudaMemcpyAsync(d_bf16, src, need, cudaMemcpyDeviceToDevice, m->stream));
  return QZO_OK;
}

int qzo_set_scales(qzo_model* m, int linear_id, const void* d_bf16, size_t bytes) {
  if (!m || !d_bf16) return QZO_ERR_BAD_ARG;
  __nv_bfloat16* dst = m->scales;
  size_t need = (size_t)m->flat_entries * 2;
  if (linear_id != -1) {
    int layer = 0, linear = 0;
    if (!split_linear_id(m, linear_id, &layer, &linear)) return QZO_ERR_BAD_ARG;
    const Linear& L = m->layers[layer].lin[linear];
    dst = m->scales + L.idx_base;
    need = (size_t)ceil_div(L.K, kGroup) * L.N * 2;
  }
  if (bytes != need) return QZO_ERR_BAD_ARG;
  QZO_CUDA_TRY(cudaMemcpyAsync(dst, d_bf16, need, cudaMemcpyDeviceToDevice, m->stream));
  return QZO_OK;
}

int qzo_debug_set_status(qzo_model* m, int value) {
  if (!m || value < 0) return QZO_ERR_BAD_ARG;
  // a host-side write of the word the kernels report through: lets a test walk the error path of a
  // step without making any device-side wait expire
  QZO_CUDA_TRY(cudaMemcpyAsync(m->status, &value, sizeof(int), cudaMemcpyHostToDevice, m->stream));
  QZO_CUDA_TRY(cudaStreamSynchronize(m->stream));
  return QZO_OK;
}

int qzo_debug_set_capture(qzo_model* m, int layer) {
  if (!m || layer < -1 || layer >= m->desc.n_layers) return QZO_ERR_BAD_ARG;
  m->capture_layer = layer;
  return QZO_OK;
}

int qzo_debug_layer_output(qzo_model* m, int layer, int which, void* d_out, size_t bytes) {
  if (!m || !d_out || m->last_T <= 0) return QZO_ERR_BAD_ARG;
  if (which == 0) {
    if (layer != m->capture_layer) return QZO_ERR_BAD_ARG;
    const size_t need = (size_t)m->last_T * m->desc.d_model * 2;
    if (bytes < need) return QZO_ERR_BAD_ARG;
    QZO_CUDA_TRY(cudaMemcpyAsync(d_out, m->capture, need, cudaMemcpyDeviceToDevice, m->stream));
  } else if (which == 1) {
    const size_t need = (size_t)m->last_T * m->desc.vocab * 4;
    if (bytes < need) return QZO_ERR_BAD_ARG;
    QZO_CUDA_TRY(cudaMemcpyAsync(d_out, m->logits, need, cudaMemcpyDeviceToDevice, m->stream));
  } else {
    return QZO_ERR_BAD_ARG;
  }
  return QZO_OK;
}

int qzo_device_status(qzo_model* m, int* h_status) {
  if (!m || !h_status) return QZO_ERR_BAD_ARG;
  QZO_CUDA_TRY(cudaMemcpyAsync(h_status, m->status, sizeof(int), cudaMemcpyDeviceToHost, m->stream));
  QZO_CUDA_TRY(cudaStreamSynchronize(m->stream));
  if (*h_status & kStatusTimeout) return QZO_ERR_DEVICE_TIMEOUT;
  return (*h_status & kStatusBadToken) ? QZO_ERR_BAD_ARG : QZO_OK;
}

}  // extern "C"
