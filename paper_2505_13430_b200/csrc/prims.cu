// Small kernels of the path that are not the GEMM: Philox / normal export, the int4
// quantiser and layout conversions, and the seeded scale update.
#include "qzo_common.cuh"
#include "philox.cuh"
#include "launch.cuh"

#include <math.h>

namespace qzo {

// ---------------------------------------------------------------------------------------
// Philox words / uniforms / normals (Sec. 3.1: z is regenerated from the seed)
// ---------------------------------------------------------------------------------------
__global__ void philox_words_kernel(uint64_t seed, uint64_t block_base, int64_t n_blocks,
                                    uint32_t* __restrict__ words, float* __restrict__ uniforms) {
  const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= n_blocks) return;
  const Philox4 p = philox_block(seed, block_base + (uint64_t)b);
  reinterpret_cast<uint4*>(words)[b] = make_uint4(p.r0, p.r1, p.r2, p.r3);
  if (uniforms) {
    reinterpret_cast<float4*>(uniforms)[b] = make_float4(uniform_from_word(p.r0), uniform_from_word(p.r1),
                                                         uniform_from_word(p.r2), uniform_from_word(p.r3));
  }
}

__global__ void normals_kernel(uint64_t seed, uint64_t index_base, int64_t count, float* __restrict__ z) {
  // one thread per counter block that overlaps [index_base, index_base + count)
  const uint64_t first_block = index_base >> 2;
  const uint64_t blk = first_block + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint64_t end = index_base + (uint64_t)count;
  if ((blk << 2) >= end) return;
  float v[4];
  normals_of_block(seed, blk, v);
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    const uint64_t i = (blk << 2) + l;
    if (i >= index_base && i < end) z[i - index_base] = v[l];
  }
}

// ---------------------------------------------------------------------------------------
// Quantiser (Eq. 3, Delta = absmax / 7 per group of 128 rows and per column)
// ---------------------------------------------------------------------------------------
__global__ void quantize_int4_kernel(const float* __restrict__ w, int K, int N,
                                     uint32_t* __restrict__ packed, __nv_bfloat16* __restrict__ scales) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (n >= N) return;
  const int k0 = g * kGroup;
  const int k1 = min(k0 + kGroup, K);
  float absmax = 0.0f;
  for (int k = k0; k < k1; ++k) absmax = fmaxf(absmax, fabsf(w[(size_t)k * N + n]));
  const __nv_bfloat16 sb = __float2bfloat16_rn(__fdiv_rn(absmax, 7.0f));
  scales[(size_t)g * N + n] = sb;
  const float s = __bfloat162float(sb);
  for (int kw = k0 / 8; kw < k1 / 8; ++kw) {
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int q = 0;
      if (s != 0.0f) {
        const float r = rintf(__fdiv_rn(w[(size_t)(kw * 8 + j) * N + n], s));   // ties to even
        q = (int)fminf(fmaxf(r, -8.0f), 7.0f);
      }
      word |= (uint32_t)(q + 8) << (4 * j);
    }
    packed[(size_t)kw * N + n] = word;
  }
}

__global__ void unpack_int4_kernel(const uint32_t* __restrict__ packed, int K, int N, int8_t* __restrict__ q) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // one packed word
  const int64_t total = (int64_t)(K / 8) * N;
  if (idx >= total) return;
  const int kw = (int)(idx / N), n = (int)(idx % N);
  const uint32_t word = packed[idx];
#pragma unroll
  for (int j = 0; j < 8; ++j) q[(size_t)(kw * 8 + j) * N + n] = (int8_t)((int)((word >> (4 * j)) & 0xF) - 8);
}

// ---------------------------------------------------------------------------------------
// Kernel layout of the packed weights.
//   block (nt, kb) = 4096 bytes at ((nt * KB + kb) * 4096), KB = ceil(K / 64);
//   inside: 16-byte unit (h * 128 + r), h = half of the k-block (32 k each), r = row in tile;
//   word i of the unit covers k = 64 kb + 32 h + 8 i .. + 7; its nibble p holds
//   k offset 2p (p < 4) or 2(p-4)+1 (p >= 4), so that ((word >> 4p) & 0x000F000F) is the
//   pair (k = 2p, 2p+1) in the low / high half.  Padding (n >= N, k >= K) is nibble 8 (q = 0).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t interleave_nibbles(uint32_t w) {
  uint32_t out = 0;
#pragma unroll
  for (int p = 0; p < 8; ++p) {
    const int src = (p < 4) ? 2 * p : 2 * (p - 4) + 1;
    out |= ((w >> (4 * src)) & 0xFu) << (4 * p);
  }
  return out;
}
__device__ __forceinline__ uint32_t deinterleave_nibbles(uint32_t w) {
  uint32_t out = 0;
#pragma unroll
  for (int p = 0; p < 8; ++p) {
    const int src = (p < 4) ? 2 * p : 2 * (p - 4) + 1;
    out |= ((w >> (4 * p)) & 0xFu) << (4 * src);
  }
  return out;
}

__global__ void repack_int4_kernel(const uint32_t* __restrict__ packed, int K, int N, uint32_t* __restrict__ out,
                                   int64_t total_words) {
  const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= total_words) return;
  const int KB = (K + kBlockK - 1) / kBlockK;
  const int i = (int)(o & 3);
  const int unit = (int)((o >> 2) & 255);
  const int64_t blk = o >> 10;
  const int kb = (int)(blk % KB);
  const int nt = (int)(blk / KB);
  const int h = unit >> 7, r = unit & 127;
  const int n = nt * kTileN + r;
  const int kw = kb * 8 + h * 4 + i;
  uint32_t w = 0x88888888u;
  if (n < N && kw < K / 8) w = packed[(size_t)kw * N + n];
  out[o] = interleave_nibbles(w);
}

__global__ void unpack_kernel_layout_kernel(const uint32_t* __restrict__ wq, int K, int N, int8_t* __restrict__ q,
                                            int64_t total_words) {
  const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= total_words) return;
  const int KB = (K + kBlockK - 1) / kBlockK;
  const int i = (int)(o & 3);
  const int unit = (int)((o >> 2) & 255);
  const int64_t blk = o >> 10;
  const int kb = (int)(blk % KB);
  const int nt = (int)(blk / KB);
  const int h = unit >> 7, r = unit & 127;
  const int n = nt * kTileN + r;
  const int kw = kb * 8 + h * 4 + i;
  if (n >= N || kw >= K / 8) return;
  const uint32_t w = deinterleave_nibbles(wq[o]);
#pragma unroll
  for (int j = 0; j < 8; ++j) q[(size_t)(kw * 8 + j) * N + n] = (int8_t)((int)((w >> (4 * j)) & 0xF) - 8);
}

// ---------------------------------------------------------------------------------------
// Seeded scale update (Algorithm 1, last loop): s_i <- bf16(max(s_i - coef z_i, 0)),
// coef = lr * clip(g) formed once in fp32 on the host or read from the device.
// One thread per counter block = four consecutive scales.
// ---------------------------------------------------------------------------------------
__global__ void update_scales_kernel(__nv_bfloat16* __restrict__ s, int64_t count, uint64_t seed,
                                     uint64_t index_base, float coef_host, const float* __restrict__ coef_dev) {
  const float coef = coef_dev ? *coef_dev : coef_host;
  if (coef == 0.0f) return;            // d' = 0 (or a rejected step): scales stay bit-identical
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t i0 = t * 4;
  if (i0 >= count) return;
  float z[4];
  normals_of_block(seed, (index_base >> 2) + (uint64_t)t, z);
  if (i0 + 4 <= count) {
    uint2 raw = *reinterpret_cast<const uint2*>(s + i0);
    __nv_bfloat16 v[4];
    *reinterpret_cast<uint2*>(v) = raw;
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      const float nv = fmaxf(__fsub_rn(__bfloat162float(v[l]), __fmul_rn(coef, z[l])), 0.0f);
      v[l] = __float2bfloat16_rn(nv);
    }
    *reinterpret_cast<uint2*>(s + i0) = *reinterpret_cast<uint2*>(v);
  } else {
    for (int l = 0; l < 4 && i0 + l < count; ++l) {
      const float nv = fmaxf(__fsub_rn(__bfloat162float(s[i0 + l]), __fmul_rn(coef, z[l])), 0.0f);
      s[i0 + l] = __float2bfloat16_rn(nv);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Joint mode (Sec. 3.2.1, closing remark; Def. 3.1, Def. 3.2): the un-quantised tensors take plain
// SPSA with z from the same (seed, index) stream, at indices that follow the scales'.
// ---------------------------------------------------------------------------------------
// dst_i = bf16(src_i + sign_eps z_i): perturbed copy of a bf16 matrix (the lm_head), four elements per
// thread = one counter block; index_base is a multiple of 4, count a multiple of 4.
__global__ void perturb_dense_bf16_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                          int64_t count, uint64_t seed, uint64_t index_base, float sign_eps) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t i0 = t * 4;
  if (i0 >= count) return;
  float z[4];
  normals_of_block(seed, (index_base >> 2) + (uint64_t)t, z);
  const uint2 raw = *reinterpret_cast<const uint2*>(src + i0);
  __nv_bfloat16 v[4];
  *reinterpret_cast<uint2*>(v) = raw;
#pragma unroll
  for (int l = 0; l < 4; ++l) v[l] = __float2bfloat16_rn(fmaf(sign_eps, z[l], __bfloat162float(v[l])));
  *reinterpret_cast<uint2*>(dst + i0) = *reinterpret_cast<uint2*>(v);
}

// Perturbed copies of a set of fp32 vectors of length d (norm gains and biases): plus[v][j] = w + eps z,
// minus[v][j] = w - eps z; src and base are device tables with one entry per vector.  grid = (ceil(d/4/256), n_vec).
__global__ void perturb_vectors_kernel(const float* const* __restrict__ src, const unsigned long long* __restrict__ base,
                                       int d, uint64_t seed, float eps, float* __restrict__ plus,
                                       float* __restrict__ minus) {
  const int v = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int j0 = t * 4;
  if (j0 >= d) return;
  float z[4];
  normals_of_block(seed, (base[v] >> 2) + (uint64_t)t, z);
  const float4 w = *reinterpret_cast<const float4*>(src[v] + j0);
  *reinterpret_cast<float4*>(plus + (size_t)v * d + j0) =
      make_float4(fmaf(eps, z[0], w.x), fmaf(eps, z[1], w.y), fmaf(eps, z[2], w.z), fmaf(eps, z[3], w.w));
  *reinterpret_cast<float4*>(minus + (size_t)v * d + j0) =
      make_float4(fmaf(-eps, z[0], w.x), fmaf(-eps, z[1], w.y), fmaf(-eps, z[2], w.z), fmaf(-eps, z[3], w.w));
}

// ZO-SGD on an un-quantised bf16 matrix: theta_i <- bf16(theta_i - coef z_i); no clamp.
__global__ void update_dense_bf16_kernel(__nv_bfloat16* __restrict__ th, int64_t count, uint64_t seed,
                                         uint64_t index_base, const float* __restrict__ coef_dev) {
  const float coef = *coef_dev;
  if (coef == 0.0f) return;
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t i0 = t * 4;
  if (i0 >= count) return;
  float z[4];
  normals_of_block(seed, (index_base >> 2) + (uint64_t)t, z);
  __nv_bfloat16 v[4];
  *reinterpret_cast<uint2*>(v) = *reinterpret_cast<const uint2*>(th + i0);
#pragma unroll
  for (int l = 0; l < 4; ++l) v[l] = __float2bfloat16_rn(__fsub_rn(__bfloat162float(v[l]), __fmul_rn(coef, z[l])));
  *reinterpret_cast<uint2*>(th + i0) = *reinterpret_cast<uint2*>(v);
}

// The same for a set of fp32 vectors (device tables as in perturb_vectors_kernel).
__global__ void update_vectors_kernel(float* const* __restrict__ th, const unsigned long long* __restrict__ base, int d,
                                      uint64_t seed, const float* __restrict__ coef_dev) {
  const float coef = *coef_dev;
  if (coef == 0.0f) return;
  const int v = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int j0 = t * 4;
  if (j0 >= d) return;
  float z[4];
  normals_of_block(seed, (base[v] >> 2) + (uint64_t)t, z);
  float4 w = *reinterpret_cast<const float4*>(th[v] + j0);
  w.x = __fsub_rn(w.x, __fmul_rn(coef, z[0])); w.y = __fsub_rn(w.y, __fmul_rn(coef, z[1]));
  w.z = __fsub_rn(w.z, __fmul_rn(coef, z[2])); w.w = __fsub_rn(w.w, __fmul_rn(coef, z[3]));
  *reinterpret_cast<float4*>(th[v] + j0) = w;
}

// ---------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------
int launch_perturb_dense_bf16(const __nv_bfloat16* src, __nv_bfloat16* dst, int64_t count, uint64_t seed,
                              uint64_t index_base, float sign_eps, cudaStream_t st) {
  if (count == 0) return QZO_OK;
  if ((count % 4) || (index_base % 4)) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(perturb_dense_bf16_kernel, dim3((unsigned)ceil_div64(count / 4, 256)), dim3(256), 0, st, src, dst, count, seed,
             index_base, sign_eps);
  return QZO_OK;
}
int launch_perturb_vectors(const float* const* src_table, const unsigned long long* base_table, int n_vec, int d,
                           uint64_t seed, float eps, float* plus, float* minus, cudaStream_t st) {
  if (n_vec == 0) return QZO_OK;
  if (d % 4) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(perturb_vectors_kernel, dim3(ceil_div(d / 4, 256), n_vec), dim3(256), 0, st, src_table, base_table, d, seed, eps,
             plus, minus);
  return QZO_OK;
}
int launch_update_dense_bf16(__nv_bfloat16* th, int64_t count, uint64_t seed, uint64_t index_base, const float* coef_dev,
                             cudaStream_t st) {
  if (count == 0) return QZO_OK;
  if ((count % 4) || (index_base % 4)) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(update_dense_bf16_kernel, dim3((unsigned)ceil_div64(count / 4, 256)), dim3(256), 0, st, th, count, seed,
             index_base, coef_dev);
  return QZO_OK;
}
int launch_update_vectors(float* const* table, const unsigned long long* base_table, int n_vec, int d, uint64_t seed,
                          const float* coef_dev, cudaStream_t st) {
  if (n_vec == 0) return QZO_OK;
  if (d % 4) return QZO_ERR_BAD_ARG;
  QZO_LAUNCH(update_vectors_kernel, dim3(ceil_div(d / 4, 256), n_vec), dim3(256), 0, st, table, base_table, d, seed, coef_dev);
  return QZO_OK;
}

int launch_philox_words(uint64_t seed, uint64_t block_base, int64_t n_blocks, uint32_t* d_words,
                        float* d_uniforms, cudaStream_t st) {
  if (n_blocks == 0) return QZO_OK;
  const int threads = 256;
  QZO_LAUNCH(philox_words_kernel, dim3((unsigned)ceil_div64(n_blocks, threads)), dim3(threads), 0, st,
             seed, block_base, n_blocks, d_words, d_uniforms);
  return QZO_OK;
}

int launch_normals(uint64_t seed, uint64_t index_base, int64_t count, float* d_z, cudaStream_t st) {
  if (count == 0) return QZO_OK;
  const int64_t n_blocks = (int64_t)(((index_base + count + 3) >> 2) - (index_base >> 2));
  const int threads = 256;
  QZO_LAUNCH(normals_kernel, dim3((unsigned)ceil_div64(n_blocks, threads)), dim3(threads), 0, st,
             seed, index_base, count, d_z);
  return QZO_OK;
}

int launch_quantize(const float* d_w, int K, int N, uint32_t* d_packed, __nv_bfloat16* d_scales, cudaStream_t st) {
  const int threads = 128;
  QZO_LAUNCH(quantize_int4_kernel, dim3(ceil_div(N, threads), ceil_div(K, kGroup)), dim3(threads), 0, st,
             d_w, K, N, d_packed, d_scales);
  return QZO_OK;
}

int launch_unpack(const uint32_t* d_packed, int K, int N, int8_t* d_q, cudaStream_t st) {
  const int64_t total = (int64_t)(K / 8) * N;
  if (total == 0) return QZO_OK;
  QZO_LAUNCH(unpack_int4_kernel, dim3((unsigned)ceil_div64(total, 256)), dim3(256), 0, st, d_packed, K, N, d_q);
  return QZO_OK;
}

size_t repacked_bytes(int K, int N) {
  return (size_t)ceil_div(N, kTileN) * ceil_div(K, kBlockK) * kPackedTileBytes;
}

int launch_repack(const uint32_t* d_packed, int K, int N, void* d_out, cudaStream_t st) {
  const int64_t words = (int64_t)(repacked_bytes(K, N) / 4);
  if (words == 0) return QZO_OK;
  QZO_LAUNCH(repack_int4_kernel, dim3((unsigned)ceil_div64(words, 256)), dim3(256), 0, st,
             d_packed, K, N, reinterpret_cast<uint32_t*>(d_out), words);
  return QZO_OK;
}

int launch_unpack_kernel_layout(const void* d_wq, int K, int N, int8_t* d_q, cudaStream_t st) {
  const int64_t words = (int64_t)(repacked_bytes(K, N) / 4);
  if (words == 0) return QZO_OK;
  QZO_LAUNCH(unpack_kernel_layout_kernel, dim3((unsigned)ceil_div64(words, 256)), dim3(256), 0, st,
             reinterpret_cast<const uint32_t*>(d_wq), K, N, d_q, words);
  return QZO_OK;
}

int launch_update_scales(__nv_bfloat16* d_s, int64_t count, uint64_t seed, uint64_t index_base,
                         float coef_host, const float* coef_dev, cudaStream_t st) {
  if (count == 0) return QZO_OK;
  const int64_t threads_total = ceil_div64(count, 4);
  QZO_LAUNCH(update_scales_kernel, dim3((unsigned)ceil_div64(threads_total, 256)), dim3(256), 0, st,
             d_s, count, seed, index_base, coef_host, coef_dev);
  return QZO_OK;
}

}  // namespace qzo
