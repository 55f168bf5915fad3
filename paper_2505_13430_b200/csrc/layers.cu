// The plain (non-GEMM) kernels of the decoder forward: embedding, RMSNorm / LayerNorm,
// RoPE, causal attention, MLP activations, fused cross entropy, and the scalar kernel that
// forms d and d' (Algorithm 1; Eq. 6).  All arithmetic is fp32 on bf16 storage.
#include "qzo_common.cuh"
#include "philox.cuh"
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
// A token id outside [0, vocab) sets bit 1 of the status word (the step then reports a bad argument and
// leaves the scales alone); the row is still written, from the nearest valid id, so nothing is read
// out of bounds.
// Joint mode (pert.sign_eps != 0): the embedding row is perturbed as E + sign eps z (Def. 3.1) with z at
// index pert.base + tok * d + j; rows from pert.pair_rows on (the second copy of a paired step) take -eps.
struct EmbedPerturb { unsigned long long seed, base; float sign_eps; int pair_rows; };

__global__ void embedding_kernel(const int32_t* __restrict__ tokens, const __nv_bfloat16* __restrict__ embed,
                                 const __nv_bfloat16* __restrict__ pos, int S, int d, int vocab,
                                 __nv_bfloat16* __restrict__ x, int* __restrict__ status, EmbedPerturb pert) {
  const int t = blockIdx.x;
  int tok = tokens[t];
  if ((tok < 0 || tok >= vocab) && threadIdx.x == 0 && status != nullptr) atomicOr(status, kStatusBadToken);
  tok = min(max(tok, 0), vocab - 1);
  const uint2* e = reinterpret_cast<const uint2*>(embed + (size_t)tok * d);
  const uint2* pp = pos ? reinterpret_cast<const uint2*>(pos + (size_t)(t % S) * d) : nullptr;
  uint2* o = reinterpret_cast<uint2*>(x + (size_t)t * d);
  const float se = (pert.pair_rows > 0 && t >= pert.pair_rows) ? -pert.sign_eps : pert.sign_eps;
  for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {       // four elements = one counter block (d % 8 == 0)
    uint2 raw = e[i];
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    if (se != 0.0f) {
      float z[4];
      normals_of_block(pert.seed, (pert.base + (unsigned long long)tok * (unsigned long long)d) / 4 + (unsigned long long)i, z);
      a.x = fmaf(se, z[0], a.x); a.y = fmaf(se, z[1], a.y); b.x = fmaf(se, z[2], b.x); b.y = fmaf(se, z[3], b.y);
    }
    if (pp) {
      const uint2 praw = pp[i];
      const __nv_bfloat162* ph = reinterpret_cast<const __nv_bfloat162*>(&praw);
      const float2 c = __bfloat1622float2(ph[0]), e2 = __bfloat1622float2(ph[1]);
      a.x += c.x; a.y += c.y; b.x += e2.x; b.y += e2.y;
    }
    __nv_bfloat162 out[2] = {__floats2bfloat162_rn(a.x, a.y), __floats2bfloat162_rn(b.x, b.y)};
    o[i] = *reinterpret_cast<const uint2*>(out);
  }
}

// Row-wise norms, optionally fused with the residual add that precedes them:
//   if delta != null:  x <- bf16(x + delta)   (the residual stream, updated in place)
//   RMSNorm:   y = x * rsqrt(mean(x^2) + eps) * w
//   LayerNorm: y = (x - mean) * rsqrt(var + eps) * w + b
// One CTA per row; the row lives in registers between the statistics and the output (16-byte
// accesses, d a multiple of 8, up to kNormVecs * 256 * 8 elements per row).  y may alias delta.
constexpr int kNormThreads = 256;
constexpr int kNormVecs = 4;

template <bool LAYERNORM>
__global__ void __launch_bounds__(kNormThreads)
add_norm_kernel(__nv_bfloat16* __restrict__ x, const __nv_bfloat16* delta, const float* __restrict__ w,
                const float* __restrict__ b, const float* __restrict__ w2, const float* __restrict__ b2, int pair_rows,
                float eps, int d, __nv_bfloat16* y) {
  // rows from pair_rows on (second copy of a paired step in joint mode) use the second gain / bias set
  if (pair_rows > 0 && (int)blockIdx.x >= pair_rows) { w = w2; b = b2; }
  __shared__ float red[32];
  const int nvec = d >> 3;
  uint4* xrow = reinterpret_cast<uint4*>(x + (size_t)blockIdx.x * d);
  const uint4* drow = delta ? reinterpret_cast<const uint4*>(delta + (size_t)blockIdx.x * d) : nullptr;
  float v[kNormVecs][8];
  float s = 0.0f;
#pragma unroll
  for (int j = 0; j < kNormVecs; ++j) {
    const int i = threadIdx.x + j * kNormThreads;
    if (i < nvec) {
      uint4 raw = xrow[i];
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
      if (drow) {
        const uint4 dr = drow[i];
        const __nv_bfloat162* dh = reinterpret_cast<const __nv_bfloat162*>(&dr);
        __nv_bfloat162 o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 a = __bfloat1622float2(h[e]), c = __bfloat1622float2(dh[e]);
          o[e] = __floats2bfloat162_rn(a.x + c.x, a.y + c.y);
          const float2 r = __bfloat1622float2(o[e]);
          v[j][2 * e] = r.x; v[j][2 * e + 1] = r.y;
        }
        xrow[i] = *reinterpret_cast<const uint4*>(o);
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 a = __bfloat1622float2(h[e]);
          v[j][2 * e] = a.x; v[j][2 * e + 1] = a.y;
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) s += LAYERNORM ? v[j][e] : v[j][e] * v[j][e];
    }
  }
  float mu = 0.0f, r;
  if (LAYERNORM) {
    mu = block_sum(s, red) / (float)d;
    float ss = 0.0f;
#pragma unroll
    for (int j = 0; j < kNormVecs; ++j) {
      if (threadIdx.x + j * kNormThreads < nvec) {
#pragma unroll
        for (int e = 0; e < 8; ++e) { const float c = v[j][e] - mu; ss += c * c; }
      }
    }
    r = rsqrtf(block_sum(ss, red) / (float)d + eps);
  } else {
    r = rsqrtf(block_sum(s, red) / (float)d + eps);
  }
  uint4* yrow = reinterpret_cast<uint4*>(y + (size_t)blockIdx.x * d);
#pragma unroll
  for (int j = 0; j < kNormVecs; ++j) {
    const int i = threadIdx.x + j * kNormThreads;
    if (i < nvec) {
      const float4 w0 = reinterpret_cast<const float4*>(w)[2 * i], w1 = reinterpret_cast<const float4*>(w)[2 * i + 1];
      const float ww[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
      float bb[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      if (LAYERNORM) {
        const float4 b0 = reinterpret_cast<const float4*>(b)[2 * i], b1 = reinterpret_cast<const float4*>(b)[2 * i + 1];
        bb[0] = b0.x; bb[1] = b0.y; bb[2] = b0.z; bb[3] = b0.w; bb[4] = b1.x; bb[5] = b1.y; bb[6] = b1.z; bb[7] = b1.w;
      }
      __nv_bfloat162 o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e)
        o[e] = __floats2bfloat162_rn((v[j][2 * e] - mu) * r * ww[2 * e] + bb[2 * e],
                                     (v[j][2 * e + 1] - mu) * r * ww[2 * e + 1] + bb[2 * e + 1]);
      yrow[i] = *reinterpret_cast<const uint4*>(o);
    }
  }
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

// Rotate pairs (i, i + dh/2) of q and k, in place.  q at buf[t][h*dh + .] with row stride ldq, k
// likewise.  One thread rotates eight consecutive pairs of one head of q or of k (16-byte accesses).
__global__ void rope_kernel(__nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k, int ldq, int ldk,
                            const float* __restrict__ cs, int S, int H, int dh, int64_t total) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int half = dh / 2;
  const int vecs = half / 8;                       // 8-pair groups per head
  const int v = (int)(idx % vecs);
  const int h = (int)((idx / vecs) % H);
  const int which = (int)((idx / ((int64_t)vecs * H)) & 1);
  const int t = (int)(idx / ((int64_t)vecs * H * 2));
  const int pos = t % S;
  __nv_bfloat16* p = (which ? k + (size_t)t * ldk : q + (size_t)t * ldq) + h * dh + v * 8;
  uint4 lo = *reinterpret_cast<const uint4*>(p), hi = *reinterpret_cast<const uint4*>(p + half);
  __nv_bfloat162* a2 = reinterpret_cast<__nv_bfloat162*>(&lo);
  __nv_bfloat162* b2 = reinterpret_cast<__nv_bfloat162*>(&hi);
  const float4* c4 = reinterpret_cast<const float4*>(cs + 2 * ((size_t)pos * half + v * 8));   // {cos, sin} pairs
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float4 cs01 = c4[e];                     // cos0 sin0 cos1 sin1
    const float2 a = __bfloat1622float2(a2[e]), b = __bfloat1622float2(b2[e]);
    a2[e] = __floats2bfloat162_rn(a.x * cs01.x - b.x * cs01.y, a.y * cs01.z - b.y * cs01.w);
    b2[e] = __floats2bfloat162_rn(b.x * cs01.x + a.x * cs01.y, b.y * cs01.z + a.y * cs01.w);
  }
  *reinterpret_cast<uint4*>(p) = lo;
  *reinterpret_cast<uint4*>(p + half) = hi;
}

// Causal attention with online softmax on the legacy tensor-core path (mma.sync m16n8k16,
// bf16 in, fp32 accumulate).  Attention is ~0.5 % of a step's FLOPs, so it stays off the
// tcgen05 path.
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float c[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// 16-byte asynchronous copy global -> shared; bytes = 0 fills the destination with zeros.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One CTA = 128 queries of one (batch, head), eight warps of 16 query rows each; keys are walked in
// blocks of 64 up to the diagonal, K and V blocks double-buffered with cp.async.  Query blocks are
// scheduled from the last (most key blocks) to the first.
constexpr int kAttBQ = 128, kAttBK = 64, kAttThreads = 256;

template <int DH>
__global__ void __launch_bounds__(kAttThreads, 2)
attention_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, int ldq, int ldk, int ldv,
                     __nv_bfloat16* __restrict__ out, int ldo, int S, float scale_log2e) {
  constexpr int BQ = kAttBQ, BK = kAttBK;
  constexpr int LD = DH + 8;                       // padded row (bf16 elements): conflict-free ldmatrix
  constexpr int CH = DH / 8;                       // 16-byte chunks per row
  extern __shared__ __align__(16) uint8_t att_smem[];
  __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(att_smem);
  __nv_bfloat16* sKV = sQ + BQ * LD;               // [2 buffers][K | V][BK][LD]

  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const size_t tok_base = (size_t)b * S;
  const int q0 = qb * BQ;
  const int last_q = min(q0 + BQ, S) - 1;
  const int nkb = last_q / BK + 1;                 // key blocks up to the diagonal of the last query row

  auto load_rows = [&](__nv_bfloat16* dst, const __nv_bfloat16* src, int ld, int row0, int rows) {
    for (int i = threadIdx.x; i < rows * CH; i += kAttThreads) {
      const int r = i / CH, c = i % CH;
      const bool in = row0 + r < S;
      const __nv_bfloat16* gp = src + (tok_base + (in ? row0 + r : 0)) * ld + h * DH + c * 8;
      cp_async16((uint32_t)__cvta_generic_to_shared(dst + r * LD + c * 8), gp, in ? 16 : 0);
    }
  };
  auto load_kv = [&](int buf, int kb) {
    __nv_bfloat16* dk = sKV + (size_t)buf * 2 * BK * LD;
    load_rows(dk, k, ldk, kb * BK, BK);
    load_rows(dk + BK * LD, v, ldv, kb * BK, BK);
  };
  load_rows(sQ, q, ldq, q0, BQ);
  load_kv(0, 0);
  cp_async_commit();
  if (nkb > 1) load_kv(1, 1);
  cp_async_commit();
  cp_async_wait<1>();                              // Q and the first K/V block have landed
  __syncthreads();

  // the Q fragments of this warp's 16 rows are re-read from shared memory in every key block
  // (keeping them in registers would cost a second resident CTA per SM)
  const int qfrag_row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.0f, l1 = 0.0f;      // rows g and g + 8 of the warp's 16
  const int qrow0 = q0 + warp * 16 + g, qrow1 = qrow0 + 8;
  const int warp_last_q = q0 + warp * 16 + 15;

  for (int kb = 0; kb < nkb; ++kb) {
    const __nv_bfloat16* sK = sKV + (size_t)(kb & 1) * 2 * BK * LD;
    const __nv_bfloat16* sV = sK + BK * LD;
    if (kb * BK <= warp_last_q) {                   // warp-uniform: this key block reaches the warp's rows
      // scores: 16 x 64 per warp
      float sc[BK / 8][4];
#pragma unroll
      for (int j = 0; j < BK / 8; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.0f;
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        uint32_t qf[4];
        ldmatrix_x4((uint32_t)__cvta_generic_to_shared(sQ + qfrag_row * LD + kk * 16 + (lane >> 4) * 8),
                    qf[0], qf[1], qf[2], qf[3]);
#pragma unroll
        for (int jp = 0; jp < BK / 16; ++jp) {      // two n8 tiles (16 keys) per ldmatrix.x4
          uint32_t b00, b01, b10, b11;
          const int key = jp * 16 + (lane & 7) + (lane >> 4) * 8;
          const int col = kk * 16 + ((lane >> 3) & 1) * 8;
          ldmatrix_x4((uint32_t)__cvta_generic_to_shared(sK + key * LD + col), b00, b01, b10, b11);
          mma_bf16_16816(sc[2 * jp], qf, b00, b01);
          mma_bf16_16816(sc[2 * jp + 1], qf, b10, b11);
        }
      }
      // causal mask (only blocks that reach past the warp's first row can cross it)
      if (kb * BK + BK - 1 > q0 + warp * 16) {
#pragma unroll
        for (int j = 0; j < BK / 8; ++j) {
          const int key = kb * BK + j * 8 + 2 * t4;
          if (key > qrow0) sc[j][0] = -INFINITY;
          if (key + 1 > qrow0) sc[j][1] = -INFINITY;
          if (key > qrow1) sc[j][2] = -INFINITY;
          if (key + 1 > qrow1) sc[j][3] = -INFINITY;
        }
      }
      // online softmax (base-2 exponent with the 1/sqrt(dh) scale folded in)
      float mx0 = m0, mx1 = m1;
#pragma unroll
      for (int j = 0; j < BK / 8; ++j) {
        mx0 = fmaxf(mx0, fmaxf(sc[j][0], sc[j][1]));
        mx1 = fmaxf(mx1, fmaxf(sc[j][2], sc[j][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float corr0 = exp2f((m0 - mx0) * scale_log2e), corr1 = exp2f((m1 - mx1) * scale_log2e);
      m0 = mx0; m1 = mx1;
      float rs0 = 0.0f, rs1 = 0.0f;
      uint32_t pf[BK / 16][4];
#pragma unroll
      for (int j = 0; j < BK / 8; ++j) {
        const float p0 = exp2f((sc[j][0] - mx0) * scale_log2e), p1 = exp2f((sc[j][1] - mx0) * scale_log2e);
        const float p2 = exp2f((sc[j][2] - mx1) * scale_log2e), p3 = exp2f((sc[j][3] - mx1) * scale_log2e);
        rs0 += p0 + p1; rs1 += p2 + p3;
        pf[j >> 1][(j & 1) * 2] = pack_bf16x2(p0, p1);
        pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16x2(p2, p3);
      }
      l0 = l0 * corr0 + rs0; l1 = l1 * corr1 + rs1;
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) { o[i][0] *= corr0; o[i][1] *= corr0; o[i][2] *= corr1; o[i][3] *= corr1; }
      // O += P V
#pragma unroll
      for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
        for (int np = 0; np < DH / 16; ++np) {      // two n8 tiles of the head dimension per ldmatrix.x4.trans
          uint32_t b00, b01, b10, b11;
          const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int col = np * 16 + (lane >> 4) * 8;
          ldmatrix_x4_trans((uint32_t)__cvta_generic_to_shared(sV + key * LD + col), b00, b01, b10, b11);
          mma_bf16_16816(o[2 * np], pf[kk], b00, b01);
          mma_bf16_16816(o[2 * np + 1], pf[kk], b10, b11);
        }
      }
    }
    __syncthreads();                                // every warp is done with buffer kb & 1
    if (kb + 2 < nkb) load_kv(kb & 1, kb + 2);
    cp_async_commit();
    cp_async_wait<1>();                             // block kb + 1 has landed (for this thread's copies)
    __syncthreads();
  }
  // normalise and store
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float inv0 = 1.0f / l0, inv1 = 1.0f / l1;
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    const int col = h * DH + i * 8 + 2 * t4;
    if (qrow0 < S)
      *reinterpret_cast<uint32_t*>(out + (tok_base + qrow0) * ldo + col) = pack_bf16x2(o[i][0] * inv0, o[i][1] * inv0);
    if (qrow1 < S)
      *reinterpret_cast<uint32_t*>(out + (tok_base + qrow1) * ldo + col) = pack_bf16x2(o[i][2] * inv1, o[i][3] * inv1);
  }
}

// act = silu(gate) * up, eight elements per thread (n is a multiple of 8)
__global__ void silu_mul_kernel(const __nv_bfloat16* __restrict__ gate, const __nv_bfloat16* __restrict__ up,
                                __nv_bfloat16* __restrict__ out, int64_t nvec) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= nvec) return;
  const uint4 g4 = reinterpret_cast<const uint4*>(gate)[i], u4 = reinterpret_cast<const uint4*>(up)[i];
  const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&g4);
  const __nv_bfloat162* u2 = reinterpret_cast<const __nv_bfloat162*>(&u4);
  __nv_bfloat162 o[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 g = __bfloat1622float2(g2[e]), u = __bfloat1622float2(u2[e]);
    o[e] = __floats2bfloat162_rn(g.x / (1.0f + __expf(-g.x)) * u.x, g.y / (1.0f + __expf(-g.y)) * u.y);
  }
  reinterpret_cast<uint4*>(out)[i] = *reinterpret_cast<const uint4*>(o);
}

__global__ void relu_kernel(__nv_bfloat16* __restrict__ x, int64_t nvec) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= nvec) return;
  uint4 v = reinterpret_cast<uint4*>(x)[i];
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
  const __nv_bfloat162 zero = __floats2bfloat162_rn(0.0f, 0.0f);
#pragma unroll
  for (int e = 0; e < 4; ++e) h[e] = __hmax2(h[e], zero);
  reinterpret_cast<uint4*>(x)[i] = v;
}

// Row-wise cross entropy on fp32 logits: row_loss[t] = logsumexp(logits[t]) - logits[t][label],
// 0 and not counted when label == -100.  One pass over the row: every thread keeps a running
// maximum and a sum of exponentials relative to it (16-byte loads when V is a multiple of 4), the
// block then merges the (max, sum) pairs in a fixed order.
__global__ void __launch_bounds__(256)
ce_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ labels, int V,
               float* __restrict__ row_loss) {
  __shared__ float red[32];
  const int t = blockIdx.x;
  const int label = labels[t];
  if (label < 0 || label >= V) {           // ignored position (uniform over the block)
    if (threadIdx.x == 0) row_loss[t] = 0.0f;
    return;
  }
  const float* row = logits + (size_t)t * V;
  float mx = -INFINITY, se = 0.0f;
  auto take = [&](float x) {
    if (x > mx) { se = se * __expf(mx - x) + 1.0f; mx = x; }
    else se += __expf(x - mx);
  };
  if ((V & 3) == 0) {
    const float4* row4 = reinterpret_cast<const float4*>(row);
    for (int i = threadIdx.x; i < (V >> 2); i += blockDim.x) {
      const float4 v = row4[i];
      take(v.x); take(v.y); take(v.z); take(v.w);
    }
  } else {
    for (int i = threadIdx.x; i < V; i += blockDim.x) take(row[i]);
  }
  const float gmx = block_max(mx, red);
  const float part = (mx == -INFINITY) ? 0.0f : se * __expf(mx - gmx);
  const float total = block_sum(part, red);
  if (threadIdx.x == 0) row_loss[t] = (gmx + logf(total)) - row[label];
}

// loss = sum(row_loss over kept rows) / count, summed in a fixed order by one block; the sum and the
// count are also written (sum_out, count_out may be null): they are what data-parallel ranks exchange.
__global__ void ce_mean_kernel(const float* __restrict__ row_loss, const int32_t* __restrict__ labels, int T, int V,
                               float* __restrict__ loss, float* __restrict__ sum_out, float* __restrict__ count_out) {
  __shared__ float red[32];
  float s = 0.0f, c = 0.0f;
  for (int i = threadIdx.x; i < T; i += blockDim.x) {
    const int lab = labels[i];
    if (lab >= 0 && lab < V) { s += row_loss[i]; c += 1.0f; }
  }
  s = block_sum(s, red);
  c = block_sum(c, red);
  if (threadIdx.x == 0) {
    if (loss) *loss = s / fmaxf(c, 1.0f);
    if (sum_out) *sum_out = s;
    if (count_out) *count_out = c;
  }
}

// sums = {sum of token losses with +eps z, the same with -eps z, kept tokens of each pass}:
// l+- = sum / count; d = (l+ - l-) / (2 eps); d' = clip(d, -C, C) (Eq. 6); coef = lr * d', forced to 0
// (no update) when a loss is not finite or the status word reports a failed launch or a bad token.
// out = {l+, l-, d, d', coef, status word as a float, coef of the un-quantised tensors (joint mode)}
__global__ void ddc_kernel(const float* __restrict__ sums, float eps, float lr, float lr_dense, float clip,
                           const int* __restrict__ status, float* __restrict__ out) {
  const float a = sums[0] / fmaxf(sums[2], 1.0f), b = sums[1] / fmaxf(sums[3], 1.0f);
  const float d = (a - b) / (2.0f * eps);
  const float dc = fminf(fmaxf(d, -clip), clip);
  const int st = status ? *status : 0;
  const bool good = isfinite(a) && isfinite(b) && st == 0;
  out[0] = a; out[1] = b; out[2] = d; out[3] = dc;
  out[4] = good ? __fmul_rn(lr, dc) : 0.0f;
  out[5] = (float)st;
  out[6] = good ? __fmul_rn(lr_dense, dc) : 0.0f;    // joint mode: step of the un-quantised tensors
}

// The per-step quantities of a recorded forward, written before it is replayed.
__global__ void set_step_params_kernel(StepParams* __restrict__ dst, StepParams v) { *dst = v; }

}  // namespace

int launch_embedding(const int32_t* tokens, const __nv_bfloat16* embed, const __nv_bfloat16* pos, int T, int S, int d,
                     int vocab, __nv_bfloat16* x, int* status, uint64_t seed, uint64_t index_base, float sign_eps,
                     int pair_rows, cudaStream_t st) {
  if ((d % 8) || (index_base % 4)) return QZO_ERR_BAD_ARG;
  const EmbedPerturb pert{seed, index_base, sign_eps, pair_rows};
  QZO_LAUNCH(embedding_kernel, dim3(T), dim3(128), 0, st, tokens, embed, pos, S, d, vocab, x, status, pert);
  return QZO_OK;
}
int launch_add_rmsnorm(__nv_bfloat16* x, const __nv_bfloat16* delta, const float* w, const float* w2, int pair_rows,
                       float eps, int T, int d, __nv_bfloat16* y, cudaStream_t st) {
  if ((d % 8) || d > kNormVecs * kNormThreads * 8) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(add_norm_kernel<false>, dim3(T), dim3(kNormThreads), 0, st, x, delta, w, nullptr, w2, nullptr, pair_rows, eps, d, y);
  return QZO_OK;
}
int launch_add_layernorm(__nv_bfloat16* x, const __nv_bfloat16* delta, const float* w, const float* b, const float* w2,
                         const float* b2, int pair_rows, float eps, int T, int d, __nv_bfloat16* y, cudaStream_t st) {
  if ((d % 8) || d > kNormVecs * kNormThreads * 8) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(add_norm_kernel<true>, dim3(T), dim3(kNormThreads), 0, st, x, delta, w, b, w2, b2, pair_rows, eps, d, y);
  return QZO_OK;
}
int launch_rope_table(float* cs, int max_seq, int dh, float theta, cudaStream_t st) {
  const int total = max_seq * (dh / 2);
  QZO_LAUNCH(rope_table_kernel, dim3(ceil_div(total, 256)), dim3(256), 0, st, cs, max_seq, dh / 2, (double)theta);
  return QZO_OK;
}
int launch_rope(__nv_bfloat16* q, __nv_bfloat16* k, int ldq, int ldk, const float* cs, int T, int S, int H, int dh,
                cudaStream_t st) {
  if ((dh % 16) || (ldq % 8) || (ldk % 8)) return QZO_ERR_BAD_ARG;
  const int64_t total = (int64_t)T * 2 * H * (dh / 16);
  QZO_LAUNCH(rope_kernel, dim3((unsigned)ceil_div64(total, 256)), dim3(256), 0, st, q, k, ldq, ldk, cs, S, H, dh, total);
  return QZO_OK;
}
int launch_attention(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, int ldq, int ldk, int ldv,
                     __nv_bfloat16* out, int ldo, int B, int S, int H, int dh, cudaStream_t st) {
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)dh);
  const dim3 grid(ceil_div(S, kAttBQ), H, B);
  if ((ldq % 8) || (ldk % 8) || (ldv % 8) || (ldo % 2)) return QZO_ERR_BAD_ARG;
  if (dh == 64) {
    constexpr int smem = (kAttBQ + 4 * kAttBK) * (64 + 8) * 2;
    static std::atomic<unsigned long long> cfg{0};
    if (first_use_on_device(cfg))
      QZO_CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    QZO_LAUNCH(attention_mma_kernel<64>, grid, dim3(kAttThreads), smem, st, q, k, v, ldq, ldk, ldv, out, ldo, S, scale_log2e);
  } else if (dh == 128) {
    constexpr int smem = (kAttBQ + 4 * kAttBK) * (128 + 8) * 2;
    static std::atomic<unsigned long long> cfg{0};
    if (first_use_on_device(cfg))
      QZO_CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    QZO_LAUNCH(attention_mma_kernel<128>, grid, dim3(kAttThreads), smem, st, q, k, v, ldq, ldk, ldv, out, ldo, S, scale_log2e);
  } else {
    return QZO_ERR_BAD_ARG;
  }
  return QZO_OK;
}
int launch_silu_mul(const __nv_bfloat16* gate, const __nv_bfloat16* up, __nv_bfloat16* out, int64_t n, cudaStream_t st) {
  if (n % 8) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(silu_mul_kernel, dim3((unsigned)ceil_div64(n / 8, 256)), dim3(256), 0, st, gate, up, out, n / 8);
  return QZO_OK;
}
int launch_relu(__nv_bfloat16* x, int64_t n, cudaStream_t st) {
  if (n % 8) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(relu_kernel, dim3((unsigned)ceil_div64(n / 8, 256)), dim3(256), 0, st, x, n / 8);
  return QZO_OK;
}
int launch_cross_entropy(const float* logits, const int32_t* labels, int T, int V, float* row_loss, float* loss,
                         float* sum_out, float* count_out, cudaStream_t st) {
  QZO_LAUNCH(ce_rows_kernel, dim3(T), dim3(256), 0, st, logits, labels, V, row_loss);
  QZO_LAUNCH(ce_mean_kernel, dim3(1), dim3(1024), 0, st, row_loss, labels, T, V, loss, sum_out, count_out);
  return QZO_OK;
}
int launch_ddc(const float* sums4, float eps, float lr, float lr_dense, float clip, const int* status, float* out7,
               cudaStream_t st) {
  QZO_LAUNCH(ddc_kernel, dim3(1), dim3(1), 0, st, sums4, eps, lr, lr_dense, clip, status, out7);
  return QZO_OK;
}
int launch_set_step_params(StepParams* d_sp, uint64_t seed, float eps, cudaStream_t st) {
  QZO_LAUNCH(set_step_params_kernel, dim3(1), dim3(1), 0, st, d_sp, StepParams{seed, eps});
  return QZO_OK;
}

}  // namespace qzo
