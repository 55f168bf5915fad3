// Kernel launch wrapper: counts launches (reported by the benchmark) and turns a launch
// error into QZO_ERR_CUDA.
#pragma once
#include "qzo_common.cuh"

namespace qzo {
void count_launch();

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
}  // namespace qzo
