// Shared declarations of the library's translation units: error codes, launch checks,
// small device helpers.  Nothing here is shared with the CPU oracle.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <atomic>

#include "../../include/qzo.h"

namespace qzo {

// Last CUDA error seen by any entry point (per process; see qzo_last_cuda_error).
void set_last_cuda_error(cudaError_t e);

#define QZO_CUDA_TRY(expr)                                  \
  do {                                                      \
    cudaError_t _e = (expr);                                \
    if (_e != cudaSuccess) {                                \
      ::qzo::set_last_cuda_error(_e);                       \
      return QZO_ERR_CUDA;                                  \
    }                                                       \
  } while (0)

#define QZO_TRY(expr)                                       \
  do {                                                      \
    int _s = (expr);                                        \
    if (_s != QZO_OK) return _s;                            \
  } while (0)

// Bits of the device status word of a model (0 = nothing to report).
constexpr int kStatusTimeout = 1;    // a bounded device-side wait expired in some launch
constexpr int kStatusBadToken = 2;   // a token id outside [0, vocab) reached the embedding

// Per-step quantities of a recorded forward (a CUDA graph that is replayed): the GEMM kernels read them
// from device memory, so that one recorded launch sequence serves every seed and every eps.
struct StepParams {
  unsigned long long seed;
  float eps;
};

constexpr int kGroup = 128;          // rows of one quantisation group (paper: group 128)
constexpr int kTileN = 128;          // output features per GEMM tile (UMMA M)
constexpr int kBlockK = 64;          // K elements per pipeline stage (one 128-byte swizzle atom of bf16)
constexpr int kPackedTileBytes = kTileN * kBlockK / 2;   // 4096: one (n-tile, k-block) of packed nibbles

// True the first time it is called for the current device with this mask (one bit per device id
// below 64; beyond that always true): per-device set-up such as cudaFuncSetAttribute is done once on
// every device a process uses, not once per process.
inline bool first_use_on_device(std::atomic<unsigned long long>& mask) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
  const unsigned long long bit = 1ull << dev;
  return (mask.fetch_or(bit) & bit) == 0;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Checks that the current device is a compute-capability 10.x part; there is no other backend.
int check_device();

}  // namespace qzo
