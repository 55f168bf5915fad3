// Launchers of the non-GEMM kernels (layers.cu) and of the GEMMs (gemm_w4a16.cu).
#pragma once
#include "qzo_common.cuh"

namespace qzo {
// sign_eps != 0: rows are perturbed as E + sign_eps z(seed, index_base + tok d + j); rows from pair_rows on take -sign_eps
int launch_embedding(const int32_t* tokens, const __nv_bfloat16* embed, const __nv_bfloat16* pos, int T, int S, int d,
                     int vocab, __nv_bfloat16* x, int* status, uint64_t seed, uint64_t index_base, float sign_eps,
                     int pair_rows, cudaStream_t st);
// x <- x + delta (skipped when delta is null), then y = norm(x); y may alias delta.  pair_rows > 0: rows from
// pair_rows on use the gains (and biases) w2 (b2).
int launch_add_rmsnorm(__nv_bfloat16* x, const __nv_bfloat16* delta, const float* w, const float* w2, int pair_rows,
                       float eps, int T, int d, __nv_bfloat16* y, cudaStream_t st);
int launch_add_layernorm(__nv_bfloat16* x, const __nv_bfloat16* delta, const float* w, const float* b, const float* w2,
                         const float* b2, int pair_rows, float eps, int T, int d, __nv_bfloat16* y, cudaStream_t st);
int launch_rope_table(float* cs, int max_seq, int dh, float theta, cudaStream_t st);
int launch_rope(__nv_bfloat16* q, __nv_bfloat16* k, int ldq, int ldk, const float* cs, int T, int S, int H, int dh,
                cudaStream_t st);
int launch_attention(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, int ldq, int ldk, int ldv,
                     __nv_bfloat16* out, int ldo, int B, int S, int H, int dh, cudaStream_t st);
int launch_silu_mul(const __nv_bfloat16* gate, const __nv_bfloat16* up, __nv_bfloat16* out, int64_t n, cudaStream_t st);
int launch_relu(__nv_bfloat16* x, int64_t n, cudaStream_t st);
// loss (mean), sum_out and count_out may each be null
int launch_cross_entropy(const float* logits, const int32_t* labels, int T, int V, float* row_loss, float* loss,
                         float* sum_out, float* count_out, cudaStream_t st);
// sums4 = {sum l+, sum l-, kept tokens (+), kept tokens (-)}; out7 = {l+, l-, d, d', lr d' or 0, status, lr_dense d' or 0}
int launch_ddc(const float* sums4, float eps, float lr, float lr_dense, float clip, const int* status, float* out7,
               cudaStream_t st);
int launch_set_step_params(StepParams* d_sp, uint64_t seed, float eps, cudaStream_t st);

// gemm_w4a16.cu
constexpr int kMaxSplitTokens = 128;   // token tiles above this never split along K
int gemm_splits(int M, int K, int N);
// pair_rows > 0: the launch switches the perturbation sign at that row (see paired_rows_ok)
size_t gemm_workspace_bytes(int M, int K, int N, int pair_rows = 0);
// One linear of a grouped launch: Y = X W' (+ bias), Y bf16 [M][ldo].
constexpr int kMaxGroupedLinears = 3;
struct GemmLinear {
  const void* wq;                 // kernel-layout int4 weights [K][N]
  const __nv_bfloat16* scales;    // [G][N]
  const float* bias;              // [N] or null
  __nv_bfloat16* out;             // [M][ldo]; 16-byte aligned, ldo a multiple of 8
  int ldo, N;
  uint64_t idx_base;              // logical index of scale [0][0]
};
// pair_rows > 0: rows [0, pair_rows) take sign * eps, rows [pair_rows, M) take -sign * eps, so that one
// launch serves both passes of a step; allowed when paired_rows_ok(M, pair_rows): pair_rows in {16, 32, 64, 128} or a multiple of 256.
bool paired_rows_ok(int M, int pair_rows);
// lut16 (host pointer to 16 floats, or null): table mode, see gemm_w4a16.cu; d_sp (device, or null): seed and eps
// are read from it by the kernel instead of the arguments; channel_scales: one row of scales [N] for all k
int launch_perturbed_gemm_group(const __nv_bfloat16* d_x, int M, int K, const GemmLinear* lins, int n_lin,
                                uint64_t seed, int sign, float eps, int pair_rows, void* d_ws, size_t ws_bytes,
                                int* d_status, cudaStream_t st, const float* lut16 = nullptr,
                                const StepParams* d_sp = nullptr, bool channel_scales = false);
// Test hook: later perturbed-GEMM launches of the calling thread use this wait limit (cycles; 0 = the normal
// one) and withhold the copies of quantisation group `skip_group` of every CTA (-1 = none).
void set_gemm_wait_debug(long long limit_cycles, int skip_group);
int launch_bf16_gemm_f32out(const __nv_bfloat16* d_x, const __nv_bfloat16* d_w, float* d_out, int M, int K, int N,
                            int* d_status, cudaStream_t st);
}  // namespace qzo
