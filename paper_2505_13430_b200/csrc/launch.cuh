// Kernel launch wrapper: counts launches (reported by the benchmark) and turns a launch
// error into QZO_ERR_CUDA.
#pragma once
#include "qzo_common.cuh"

namespace qzo {
void count_launch();
void add_launches(long long n);   // kernels run by replaying a recorded step

#define QZO_LAUNCH(kernel, grid, block, smem, stream, ...)                  \
  do {                                                                      \
    kernel<<<(grid), (block), (smem), (stream)>>>(__VA_ARGS__);             \
    ::qzo::count_launch();                                                  \
    cudaError_t _le = cudaGetLastError();                                   \
    if (_le != cudaSuccess) {                                               \
      ::qzo::set_last_cuda_error(_le);                                      \
      return QZO_ERR_CUDA;                                                  \
    }                                                                       \
  } while (0)

// prims.cu
int launch_philox_words(uint64_t seed, uint64_t block_base, int64_t n_blocks, uint32_t* d_words,
                        float* d_uniforms, cudaStream_t st);
int launch_normals(uint64_t seed, uint64_t index_base, int64_t count, float* d_z, cudaStream_t st);
int launch_quantize(const float* d_w, int K, int N, uint32_t* d_packed, __nv_bfloat16* d_scales, cudaStream_t st);
int launch_unpack(const uint32_t* d_packed, int K, int N, int8_t* d_q, cudaStream_t st);
size_t repacked_bytes(int K, int N);
int launch_repack(const uint32_t* d_packed, int K, int N, void* d_out, cudaStream_t st);
int launch_unpack_kernel_layout(const void* d_wq, int K, int N, int8_t* d_q, cudaStream_t st);
int launch_update_scales(__nv_bfloat16* d_s, int64_t count, uint64_t seed, uint64_t index_base,
                         float coef_host, const float* coef_dev, cudaStream_t st);
// joint mode: plain SPSA on the un-quantised tensors
int launch_perturb_dense_bf16(const __nv_bfloat16* src, __nv_bfloat16* dst, int64_t count, uint64_t seed,
                              uint64_t index_base, float sign_eps, cudaStream_t st);
int launch_perturb_vectors(const float* const* src_table, const unsigned long long* base_table, int n_vec, int d,
                           uint64_t seed, float eps, float* plus, float* minus, cudaStream_t st);
int launch_update_dense_bf16(__nv_bfloat16* th, int64_t count, uint64_t seed, uint64_t index_base, const float* coef_dev,
                             cudaStream_t st);
int launch_update_vectors(float* const* table, const unsigned long long* base_table, int n_vec, int d, uint64_t seed,
                          const float* coef_dev, cudaStream_t st);
}  // namespace qzo
