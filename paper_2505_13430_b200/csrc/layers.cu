// The plain (non-GEMM) kernels of the decoder forward: embedding, RMSNorm / LayerNorm,
// RoPE, causal attention, MLP activations, fused cross entropy, and the scalar kernel that
// forms d and d' (Algorithm 1; Eq. 6).  All arithmetic is fp32 on bf16 storage.
#include "qzo_common.cuh"
#include "launch.cuh"
#include "layers.cuh"

#include <math.h>

namespace qzo {

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Block-wide sum with a fixed reduction tree (deterministic); blockDim.x multiple of 32, <= 1024.
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < nw) ? red[l] : 0.0f;
  return warp_sum(t);
}
__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < nw) ? red[l] : -INFINITY;
  return warp_max(t);
}

// x[t][:] = E[tok[t]][:] (+ P[t % S][:])
__global__ void embedding_kernel(const int32_t* __restrict__ tokens, const __nv_bfloat16* __restrict__ embed,
                                 const __nv_bfloat16* __restrict__ pos, int S, int d, int vocab,
                                 __nv_bfloat16* __restrict__ x) {
  const int t = blockIdx.x;
  int tok = tokens[t];
  tok = min(max(tok, 0), vocab - 1);
  const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(embed + (size_t)tok * d);
  const __nv_bfloat162* pp = pos ? reinterpret_cast<const __nv_bfloat162*>(pos + (size_t)(t % S) * d) : nullptr;
  __nv_bfloat162* o = reinterpret_cast<__nv_bfloat162*>(x + (size_t)t * d);
  for (int i = threadIdx.x; i < d / 2; i += blockDim.x) {
    float2 v = __bfloat1622float2(e[i]);
    if (pp) {
      const float2 q = __bfloat1622float2(pp[i]);
      v.x += q.x; v.y += q.y;
    }
    o[i] = __floats2bfloat162_rn(v.x, v.y);
  }
}

// y = x * rsqrt(mean(x^2) + eps) * w
__global__ void rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ w, float eps, int d,
                               __nv_bfloat16* __restrict__ y) {
  __shared__ float red[32];
  const __nv_bfloat16* row = x + (size_t)blockIdx.x * d;
  float ss = 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = __bfloat162float(row[i]);
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)d + eps);
  __nv_bfloat16* out = y + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) out[i] = __float2bfloat16_rn(__bfloat162float(row[i]) * r * w[i]);
}

// y = (x - mean) * rsqrt(var + eps) * w + b
__global__ void layernorm_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ w,
                                 const float* __restrict__ b, float eps, int d, __nv_bfloat16* __restrict__ y) {
  __shared__ float red[32];
  const __nv_bfloat16* row = x + (size_t)blockIdx.x * d;
  float s = 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) s += __bfloat162float(row[i]);
  const float mu = block_sum(s, red) / (float)d;
  float ss = 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float c = __bfloat162float(row[i]) - mu;
    ss += c * c;
  }
  const float r = rsqrtf(block_sum(ss, red) / (float)d + eps);
  __nv_bfloat16* out = y + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    out[i] = __float2bfloat16_rn((__bfloat162float(row[i]) - mu) * r * w[i] + b[i]);
}

// cos/sin table [max_seq][dh/2] in fp32, evaluated in fp64.
__global__ void rope_table_kernel(float* __restrict__ cs, int max_seq, int half, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_seq * half) return;
  const int pos = idx / half, i = idx % half;
  const double inv = pow(theta, -(double)i / (double)half);
  double s, c;
  sincos((double)pos * inv, &s, &c);
  cs[2 * idx] = (float)c;
  cs[2 * idx + 1] = (float)s;
}

// Rotate pairs (i, i + dh/2) of q and k, in place.  q at buf[t][q_off + h*dh + .], k at k_off.
__global__ void rope_kernel(__nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k, int ldq, int ldk,
                            const float* __restrict__ cs, int S, int H, int dh, int64_t total) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int half = dh / 2;
  const int i = (int)(idx % half);
  const int h = (int)((idx / half) % H);
  const int t = (int)(idx / ((int64_t)half * H));
  const int pos = t % S;
  const float c = cs[2 * (pos * half + i)], s = cs[2 * (pos * half + i) + 1];
  {
    __nv_bfloat16* p = q + (size_t)t * ldq + h * dh + i;
    const float a = __bfloat162float(p[0]), b = __bfloat162float(p[half]);
    p[0] = __float2bfloat16_rn(a * c - b * s);
    p[half] = __float2bfloat16_rn(b * c + a * s);
  }
  {
    __nv_bfloat16* p = k + (size_t)t * ldk + h * dh + i;
    const float a = __bfloat162float(p[0]), b = __bfloat162float(p[half]);
    p[0] = __float2bfloat16_rn(a * c - b * s);
    p[half] = __float2bfloat16_rn(b * c + a * s);
  }
}

// Causal attention, one warp per (batch, head, query): online softmax over keys 0..query.
// DH in {64, 128}; each lane holds DH/32 features.
template <int DH>
__global__ void attention_simple_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                        const __nv_bfloat16* __restrict__ v, int ldq, int ldk, int ldv,
                                        __nv_bfloat16* __restrict__ out, int ldo, int B, int S, int H, float scale) {
  constexpr int E = DH / 32;
  const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (int64_t)B * H * S) return;
  const int sq = (int)(wid % S);
  const int h = (int)((wid / S) % H);
  const int b = (int)(wid / ((int64_t)S * H));
  const int t = b * S + sq;
  float qv[E], acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    qv[e] = __bfloat162float(q[(size_t)t * ldq + h * DH + lane * E + e]) * scale;
    acc[e] = 0.0f;
  }
  float m = -INFINITY, l = 0.0f;
  for (int j = 0; j <= sq; ++j) {
    const size_t tk = (size_t)(b * S + j);
    float part = 0.0f;
#pragma unroll
    for (int e = 0; e < E; ++e) part += qv[e] * __bfloat162float(k[tk * ldk + h * DH + lane * E + e]);
    const float sc = warp_sum(part);
    const float mn = fmaxf(m, sc);
    const float corr = __expf(m - mn);
    const float pj = __expf(sc - mn);
    l = l * corr + pj;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + pj * __bfloat162float(v[tk * ldv + h * DH + lane * E + e]);
    m = mn;
  }
  const float inv = 1.0f / l;
#pragma unroll
  for (int e = 0; e < E; ++e) out[(size_t)t * ldo + h * DH + lane * E + e] = __float2bfloat16_rn(acc[e] * inv);
}

// act = silu(gate) * up
__global__ void silu_mul_kernel(const __nv_bfloat16* __restrict__ gate, const __nv_bfloat16* __restrict__ up,
                                __nv_bfloat16* __restrict__ out, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float g = __bfloat162float(gate[i]), u = __bfloat162float(up[i]);
  out[i] = __float2bfloat16_rn(g / (1.0f + __expf(-g)) * u);
}

__global__ void relu_kernel(__nv_bfloat16* __restrict__ x, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  x[i] = __float2bfloat16_rn(fmaxf(__bfloat162float(x[i]), 0.0f));
}

// Row-wise cross entropy on fp32 logits: row_loss[t] = logsumexp(logits[t]) - logits[t][label],
// 0 and not counted when label == -100.
__global__ void ce_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ labels, int V,
                               float* __restrict__ row_loss) {
  __shared__ float red[32];
  const int t = blockIdx.x;
  const int label = labels[t];
  if (label < 0 || label >= V) {           // ignored position (uniform over the block)
    if (threadIdx.x == 0) row_loss[t] = 0.0f;
    return;
  }
  const float* row = logits + (size_t)t * V;
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < V; i += blockDim.x) mx = fmaxf(mx, row[i]);
  mx = block_max(mx, red);
  float se = 0.0f;
  for (int i = threadIdx.x; i < V; i += blockDim.x) se += expf(row[i] - mx);
  se = block_sum(se, red);
  if (threadIdx.x == 0) row_loss[t] = (mx + logf(se)) - row[label];
}

// loss = sum(row_loss over kept rows) / count, summed in a fixed order by one block.
__global__ void ce_mean_kernel(const float* __restrict__ row_loss, const int32_t* __restrict__ labels, int T, int V,
                               float* __restrict__ loss) {
  __shared__ float red[32];
  float s = 0.0f, c = 0.0f;
  for (int i = threadIdx.x; i < T; i += blockDim.x) {
    const int lab = labels[i];
    if (lab >= 0 && lab < V) { s += row_loss[i]; c += 1.0f; }
  }
  s = block_sum(s, red);
  c = block_sum(c, red);
  if (threadIdx.x == 0) *loss = s / fmaxf(c, 1.0f);
}

// d = (l+ - l-) / (2 eps); d' = clip(d, -C, C) (Eq. 6); coef = lr * d' (0 if a loss is not finite).
// out = {l+, l-, d, d', coef}
__global__ void ddc_kernel(const float* __restrict__ lp, const float* __restrict__ lm, float eps, float lr, float clip,
                           float* __restrict__ out) {
  const float a = *lp, b = *lm;
  const float d = (a - b) / (2.0f * eps);
  const float dc = fminf(fmaxf(d, -clip), clip);
  const bool finite = isfinite(a) && isfinite(b);
  out[0] = a; out[1] = b; out[2] = d; out[3] = dc;
  out[4] = finite ? __fmul_rn(lr, dc) : 0.0f;
}

}  // namespace

int launch_embedding(const int32_t* tokens, const __nv_bfloat16* embed, const __nv_bfloat16* pos, int T, int S, int d,
                     int vocab, __nv_bfloat16* x, cudaStream_t st) {
  QZO_LAUNCH(embedding_kernel, dim3(T), dim3(128), 0, st, tokens, embed, pos, S, d, vocab, x);
  return QZO_OK;
}
int launch_rmsnorm(const __nv_bfloat16* x, const float* w, float eps, int T, int d, __nv_bfloat16* y, cudaStream_t st) {
  QZO_LAUNCH(rmsnorm_kernel, dim3(T), dim3(256), 0, st, x, w, eps, d, y);
  return QZO_OK;
}
int launch_layernorm(const __nv_bfloat16* x, const float* w, const float* b, float eps, int T, int d,
                     __nv_bfloat16* y, cudaStream_t st) {
  QZO_LAUNCH(layernorm_kernel, dim3(T), dim3(256), 0, st, x, w, b, eps, d, y);
  return QZO_OK;
}
int launch_rope_table(float* cs, int max_seq, int dh, float theta, cudaStream_t st) {
  const int total = max_seq * (dh / 2);
  QZO_LAUNCH(rope_table_kernel, dim3(ceil_div(total, 256)), dim3(256), 0, st, cs, max_seq, dh / 2, (double)theta);
  return QZO_OK;
}
int launch_rope(__nv_bfloat16* q, __nv_bfloat16* k, int ldq, int ldk, const float* cs, int T, int S, int H, int dh,
                cudaStream_t st) {
  const int64_t total = (int64_t)T * H * (dh / 2);
  QZO_LAUNCH(rope_kernel, dim3((unsigned)ceil_div64(total, 256)), dim3(256), 0, st, q, k, ldq, ldk, cs, S, H, dh, total);
  return QZO_OK;
}
int launch_attention(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, int ldq, int ldk, int ldv,
                     __nv_bfloat16* out, int ldo, int B, int S, int H, int dh, cudaStream_t st) {
  const int64_t warps = (int64_t)B * H * S;
  const float scale = 1.0f / sqrtf((float)dh);
  const dim3 grid((unsigned)ceil_div64(warps * 32, 256));
  if (dh == 64) {
    QZO_LAUNCH(attention_simple_kernel<64>, grid, dim3(256), 0, st, q, k, v, ldq, ldk, ldv, out, ldo, B, S, H, scale);
  } else if (dh == 128) {
    QZO_LAUNCH(attention_simple_kernel<128>, grid, dim3(256), 0, st, q, k, v, ldq, ldk, ldv, out, ldo, B, S, H, scale);
  } else {
    return QZO_ERR_BAD_ARG;
  }
  return QZO_OK;
}
int launch_silu_mul(const __nv_bfloat16* gate, const __nv_bfloat16* up, __nv_bfloat16* out, int64_t n, cudaStream_t st) {
  QZO_LAUNCH(silu_mul_kernel, dim3((unsigned)ceil_div64(n, 256)), dim3(256), 0, st, gate, up, out, n);
  return QZO_OK;
}
int launch_relu(__nv_bfloat16* x, int64_t n, cudaStream_t st) {
  QZO_LAUNCH(relu_kernel, dim3((unsigned)ceil_div64(n, 256)), dim3(256), 0, st, x, n);
  return QZO_OK;
}
int launch_cross_entropy(const float* logits, const int32_t* labels, int T, int V, float* row_loss, float* loss,
                         cudaStream_t st) {
  QZO_LAUNCH(ce_rows_kernel, dim3(T), dim3(256), 0, st, logits, labels, V, row_loss);
  QZO_LAUNCH(ce_mean_kernel, dim3(1), dim3(1024), 0, st, row_loss, labels, T, V, loss);
  return QZO_OK;
}
int launch_ddc(const float* lp, const float* lm, float eps, float lr, float clip, float* out5, cudaStream_t st) {
  QZO_LAUNCH(ddc_kernel, dim3(1), dim3(1), 0, st, lp, lm, eps, lr, clip, out5);
  return QZO_OK;
}

}  // namespace qzo
