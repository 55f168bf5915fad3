// Perturbed W4A16 GEMM for sm_100a: Y[t][n] = sum_k X[t][k] (s[k/128][n] + sign eps z_i) q[k][n].
//
// Eq. 4 (w = Delta * w_bar) is evaluated in the kernel's prologue with the perturbed scale
// of Eq. 5, Delta' = Delta + sign eps z, formed in fp32 from the stored bf16 scale and a
// Gaussian z regenerated from (seed, logical scale index); the stored scales are never
// written.  The contraction runs on the tcgen05 tensor cores with the accumulator in TMEM.
//
// Tile roles.  The de-quantised weight tile is the MMA's A operand (UMMA M = 128 output
// features), the activation tile is the B operand (UMMA N = TOK tokens, 16..256), so that
// one de-quantised weight feeds TOK multiply-adds and small token counts do not waste
// tensor rows.  D[n][t] sits in TMEM with lane = output feature, column = token.
//
// Warp roles (12 warps):
//   warp 0      TMA producer: activation tile (2-D tensor map, 128-byte swizzle), packed
//               int4 tile (one 4 KiB bulk copy), raw bf16 scales of a group (bulk copy)
//   warp 1      MMA issuer (one elected lane), owns the TMEM allocation
//   warps 2-3   scale warps: Philox4x32-10 + Box-Muller, s' = s + sign eps z in fp32, split
//               into bf16 hi + lo parts, written to a small shared-memory ring
//   warps 4-11  de-quantisers: nibbles -> bf16 (u - 8) * s' into the swizzled K-major
//               A tile; afterwards the epilogue (TMEM -> registers -> global)
// Every wait on an mbarrier is bounded; when a wait expires the CTA records an error in
// the status word, drains its copies and leaves through the common exit (TMEM is freed).
#include "qzo_common.cuh"
#include "philox.cuh"
#include "launch.cuh"

#include <cuda.h>
#include <mutex>

namespace qzo {

namespace {

constexpr int kStagesDequant = 6;     // pipeline depth over k-blocks, int4 path (A operand lives in TMEM)
constexpr int kStagesBf16 = 4;        // bf16-weight path (A operand tile in shared memory)
constexpr int kATmemColsPerStage = kBlockK / 2;   // 64 bf16 along K = 32 TMEM columns of 32 bits
constexpr int kScaleSlots = 4;        // ring of perturbed-scale rows (one per quantisation group)
constexpr int kNumScaleWarps = 2;
constexpr int kNumDeqWarps = 8;
constexpr int kFirstScaleWarp = 2;
constexpr int kFirstDeqWarp = 4;
constexpr int kNumWarps = kFirstDeqWarp + kNumDeqWarps;
constexpr int kThreads = kNumWarps * 32;
constexpr int kDeqThreads = kNumDeqWarps * 32;
constexpr long long kWaitLimitCycles = 4000000000LL;   // ~2 s at boost clock

constexpr int kWTileBytes = kTileN * kBlockK * 2;      // 16 KiB bf16 A tile
constexpr int kRawScaleBytes = kTileN * 2;             // 256 B
constexpr int kCookedScaleBytes = kTileN * 8;          // {hi,hi},{lo,lo} per output feature

enum OutMode { kOutBf16 = 0, kOutF32 = 1 };

struct GemmParams {
  const uint8_t* wq;              // kernel-layout int4 (dequant mode)
  const __nv_bfloat16* scales;    // [G][N] of this linear
  const float* bias;              // [N] or null
  const __nv_bfloat16* residual;  // [M][ldo] or null (added in the epilogue, may alias out)
  void* out;                      // bf16 [M][ldo]  or  float [splits][M][ldo]
  int M, K, N, ldo;
  int num_kb;                     // ceil(K / 64)
  int kb_per_split;               // even number of k-blocks per blockIdx.z
  uint64_t seed, idx_base;
  float sign_eps;                 // sign * eps (0 when unperturbed)
  int* status;
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit expired or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 0xFF) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Same MMA with the A operand read from tensor memory (lane = row, 2 bf16 per 32-bit column).
__device__ __forceinline__ void umma_bf16_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t v[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t v[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile with 128-byte swizzle: rows are
// 128 bytes, eight rows form a 1024-byte swizzle atom (stride byte offset 1024), descriptor
// version 1, layout type 2 (128-byte swizzle).  The tile base must be 1024-byte aligned; a
// 16-element step along K advances the start address by 32 bytes.
__device__ __forceinline__ uint64_t umma_desc_k_major_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // descriptor version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M x N.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ----------------------------------------------------------------------------- shared memory plan
template <int TOK, bool DEQUANT>
struct SmemPlan {
  static constexpr int kStages = DEQUANT ? kStagesDequant : kStagesBf16;
  static constexpr int kXTileBytes = TOK * kBlockK * 2;
  // int4 path: [X tile | packed nibbles]; bf16 path: [W tile | X tile]
  static constexpr int kStageBytes = DEQUANT ? (kXTileBytes + kPackedTileBytes) : (kWTileBytes + kXTileBytes);
  static constexpr int kOffW = 0;                                   // bf16 path only
  static constexpr int kOffX = DEQUANT ? 0 : kWTileBytes;
  static constexpr int kOffP = kXTileBytes;                         // int4 path only
  static constexpr int kOffRaw = kStages * kStageBytes;
  static constexpr int kOffCooked = kOffRaw + kScaleSlots * kRawScaleBytes;
  static constexpr int kOffBars = kOffCooked + kScaleSlots * kCookedScaleBytes;
  static constexpr int kNumBars = 3 * kStages + 4 * kScaleSlots + 1;
  static constexpr int kOffMisc = kOffBars + kNumBars * 8;
  static constexpr int kTotal = kOffMisc + 16;
  static constexpr int kDynamicBytes = kTotal + 1024;      // slack for the 1024-byte alignment
};

// ----------------------------------------------------------------------------- the kernel
// DEQUANT = true : A operand produced from packed int4 + perturbed scales.
// DEQUANT = false: A operand is a bf16 [N][K] row-major matrix loaded through tmap_w (lm_head).
template <int TOK, bool DEQUANT, int OUT_MODE>
__global__ void __launch_bounds__(kThreads, 1)
w4a16_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                  const GemmParams p) {
  using Plan = SmemPlan<TOK, DEQUANT>;
  constexpr int kStages = Plan::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const smem = smem_raw + (base - smem_u32(smem_raw));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  const uint32_t bar0 = base + Plan::kOffBars;
  auto bar_full = [&](int s) { return bar0 + 8u * s; };                          // TMA landed (X, packed / W)
  auto bar_deq = [&](int s) { return bar0 + 8u * (kStages + s); };              // A tile de-quantised
  auto bar_empty = [&](int s) { return bar0 + 8u * (2 * kStages + s); };        // MMAs of the stage retired
  auto bar_raw_full = [&](int g) { return bar0 + 8u * (3 * kStages + g); };
  auto bar_raw_empty = [&](int g) { return bar0 + 8u * (3 * kStages + kScaleSlots + g); };
  auto bar_sc_full = [&](int g) { return bar0 + 8u * (3 * kStages + 2 * kScaleSlots + g); };
  auto bar_sc_empty = [&](int g) { return bar0 + 8u * (3 * kStages + 3 * kScaleSlots + g); };
  const uint32_t bar_acc = bar0 + 8u * (3 * kStages + 4 * kScaleSlots);
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(smem + Plan::kOffMisc);
  uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(smem + Plan::kOffMisc + 4);
  volatile int* const never_set = reinterpret_cast<volatile int*>(smem + Plan::kOffMisc + 8);   // stays 0

  const int n0 = blockIdx.x * kTileN;
  const int tok0 = blockIdx.y * TOK;
  const int kb_begin = blockIdx.z * p.kb_per_split;
  const int kb_end = min(kb_begin + p.kb_per_split, p.num_kb);
  const int nkb = kb_end - kb_begin;                     // >= 1 by construction of the grid

  // TMEM columns: accumulator [0, TOK), then (int4 path) one 32-column A tile per stage
  constexpr uint32_t kAccCols = TOK < 32 ? 32 : TOK;
  constexpr uint32_t kUsedCols = DEQUANT ? kAccCols + kStages * kATmemColsPerStage : kAccCols;
  constexpr uint32_t kTmemCols = kUsedCols <= 32 ? 32 : kUsedCols <= 64 ? 64 : kUsedCols <= 128 ? 128
                                 : kUsedCols <= 256 ? 256 : 512;
  static_assert(kUsedCols <= 512, "TMEM budget");

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    *never_set = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_deq(s), kDeqThreads);
      mbar_init(bar_empty(s), 1);
    }
    for (int g = 0; g < kScaleSlots; ++g) {
      mbar_init(bar_raw_full(g), 1);
      mbar_init(bar_raw_empty(g), 32);
      mbar_init(bar_sc_full(g), 32);
      mbar_init(bar_sc_empty(g), kDeqThreads);
    }
    mbar_init(bar_acc, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  bool ok = true;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int issued = 0;
      for (int it = 0; it < nkb; ++it) {
        const int s = it % kStages;
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        const int kb = kb_begin + it;
        if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t stage = base + s * Plan::kStageBytes;
        if (DEQUANT) {
          mbar_arrive_expect_tx(bar_full(s), Plan::kXTileBytes + kPackedTileBytes);
          bulk_load(stage + Plan::kOffP,
                    p.wq + ((size_t)blockIdx.x * p.num_kb + kb) * kPackedTileBytes, kPackedTileBytes, bar_full(s));
        } else {
          mbar_arrive_expect_tx(bar_full(s), Plan::kXTileBytes + kWTileBytes);
          tma_load_2d(stage + Plan::kOffW, &tmap_w, bar_full(s), kb * kBlockK, n0);
        }
        tma_load_2d(stage + Plan::kOffX, &tmap_x, bar_full(s), kb * kBlockK, tok0);
        issued = it + 1;
        if (DEQUANT && ((it & 1) == 0)) {
          // first k-block of a quantisation group: fetch the group's raw scales
          const int gi = it >> 1;
          const int slot = gi % kScaleSlots;
          const uint32_t gph = (uint32_t)(gi / kScaleSlots) & 1u;
          if (!mbar_wait(bar_raw_empty(slot), gph ^ 1u, abort_flag)) { ok = false; break; }
          const int g = (kb >> 1);
          const int valid = min(kTileN, p.N - n0);
          const uint32_t bytes = (uint32_t)valid * 2u;
          mbar_arrive_expect_tx(bar_raw_full(slot), bytes);
          bulk_load(base + Plan::kOffRaw + slot * kRawScaleBytes, p.scales + (size_t)g * p.N + n0, bytes,
                    bar_raw_full(slot));
        }
      }
      if (!ok) {
        // drain: give the copies already issued a bounded chance to land before the CTA exits
        *abort_flag = 1;
        for (int it = max(0, issued - kStages); it < issued; ++it)
          mbar_wait(bar_full(it % kStages), (uint32_t)(it / kStages) & 1u, never_set);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTileN, TOK);
      for (int it = 0; it < nkb; ++it) {
        const int s = it % kStages;
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        if (!mbar_wait(bar_full(s), ph, abort_flag)) { ok = false; break; }
        if (DEQUANT) {
          if (!mbar_wait(bar_deq(s), ph, abort_flag)) { ok = false; break; }
        }
        tcgen05_fence_after();
        const uint32_t stage = base + s * Plan::kStageBytes;
        const uint64_t bdesc = umma_desc_k_major_sw128(stage + Plan::kOffX);
        if (DEQUANT) {
          const uint32_t a_tmem = tmem_d + kAccCols + (uint32_t)(s * kATmemColsPerStage);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)      // 16 bf16 along K = 8 TMEM columns
            umma_bf16_tmem_a(tmem_d, a_tmem + (uint32_t)(k * 8), bdesc + (uint64_t)(k * 2), idesc,
                             (it > 0 || k > 0) ? 1u : 0u);
        } else {
          const uint64_t adesc = umma_desc_k_major_sw128(stage + Plan::kOffW);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)
            umma_bf16(tmem_d, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                      (it > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(bar_empty(s));
      }
      if (ok) umma_commit(bar_acc);
      else *abort_flag = 1;
    }
  } else if (warp < kFirstDeqWarp) {
    // ------------------------------------------------------------------ scale warps
    if (DEQUANT) {
      const int sw = warp - kFirstScaleWarp;
      const int ngroups = (nkb + 1) >> 1;
      for (int gi = sw; gi < ngroups; gi += kNumScaleWarps) {
        const int slot = gi % kScaleSlots;
        const uint32_t gph = (uint32_t)(gi / kScaleSlots) & 1u;
        const int g = (kb_begin >> 1) + gi;
        if (!mbar_wait(bar_raw_full(slot), gph, abort_flag)) { ok = false; break; }
        const __nv_bfloat16* raw = reinterpret_cast<const __nv_bfloat16*>(smem + Plan::kOffRaw + slot * kRawScaleBytes);
        const int r0 = lane * 4;                       // four consecutive output features = one counter block
        float sv[4];
#pragma unroll
        for (int l = 0; l < 4; ++l) sv[l] = (n0 + r0 + l < p.N) ? __bfloat162float(raw[r0 + l]) : 0.0f;
        mbar_arrive(bar_raw_empty(slot));
        if (p.sign_eps != 0.0f) {
          float z[4];
          const uint64_t i0 = p.idx_base + (uint64_t)g * (uint64_t)p.N + (uint64_t)(n0 + r0);
          normals_of_block(p.seed, i0 >> 2, z);
#pragma unroll
          for (int l = 0; l < 4; ++l) sv[l] = (n0 + r0 + l < p.N) ? fmaf(p.sign_eps, z[l], sv[l]) : 0.0f;
        }
        uint32_t cooked[8];
#pragma unroll
        for (int l = 0; l < 4; ++l) {
          const __nv_bfloat16 hi = __float2bfloat16_rn(sv[l]);
          const __nv_bfloat16 lo = __float2bfloat16_rn(sv[l] - __bfloat162float(hi));
          const uint32_t h16 = (uint32_t)__bfloat16_as_ushort(hi), l16 = (uint32_t)__bfloat16_as_ushort(lo);
          cooked[2 * l] = h16 | (h16 << 16);
          cooked[2 * l + 1] = l16 | (l16 << 16);
        }
        if (!mbar_wait(bar_sc_empty(slot), gph ^ 1u, abort_flag)) { ok = false; break; }
        uint4* dst = reinterpret_cast<uint4*>(smem + Plan::kOffCooked + slot * kCookedScaleBytes + r0 * 8);
        dst[0] = make_uint4(cooked[0], cooked[1], cooked[2], cooked[3]);
        dst[1] = make_uint4(cooked[4], cooked[5], cooked[6], cooked[7]);
        mbar_arrive(bar_sc_full(slot));
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ de-quantisers, then epilogue
    const int dt = threadIdx.x - kFirstDeqWarp * 32;      // 0..255
    if (DEQUANT) {
      const int r = (warp & 3) * 32 + lane;               // row of the tile = TMEM lane this warp may access
      const int h = dt >> 7;                              // half of the k-block (32 k each)
      const __nv_bfloat162 magic_bias = __halves2bfloat162(__float2bfloat16_rn(136.0f), __float2bfloat16_rn(136.0f));
      __nv_bfloat162 s_hi, s_lo;
      *reinterpret_cast<uint32_t*>(&s_hi) = 0u;
      *reinterpret_cast<uint32_t*>(&s_lo) = 0u;
      for (int it = 0; it < nkb && ok; ++it) {
        const int s = it % kStages;
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        if ((it & 1) == 0) {
          const int gi = it >> 1;
          const int slot = gi % kScaleSlots;
          const uint32_t gph = (uint32_t)(gi / kScaleSlots) & 1u;
          if (!__all_sync(0xffffffffu, mbar_wait(bar_sc_full(slot), gph, abort_flag))) { ok = false; break; }
          const uint2 c = *reinterpret_cast<const uint2*>(smem + Plan::kOffCooked + slot * kCookedScaleBytes + r * 8);
          *reinterpret_cast<uint32_t*>(&s_hi) = c.x;
          *reinterpret_cast<uint32_t*>(&s_lo) = c.y;
          mbar_arrive(bar_sc_empty(slot));
        }
        // bar_full(s) completing implies the stage was released by the MMAs that last read it
        if (!__all_sync(0xffffffffu, mbar_wait(bar_full(s), ph, abort_flag))) { ok = false; break; }
        tcgen05_fence_after();                              // orders the MMAs' reads of this A stage before the store below
        uint8_t* stage = smem + s * Plan::kStageBytes;
        const uint4 pk = *reinterpret_cast<const uint4*>(stage + Plan::kOffP + (h * kTileN + r) * 16);
        const uint32_t words[4] = {pk.x, pk.y, pk.z, pk.w};
        uint32_t outw[16];                                  // k = 32 h + 2 j, 2 j + 1 in register j
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
          for (int pp = 0; pp < 4; ++pp) {
            uint32_t x = ((words[i] >> (4 * pp)) & 0x000F000Fu) | 0x43004300u;     // bf16x2 {128 + u_lo, 128 + u_hi}
            __nv_bfloat162 q2 = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&x), magic_bias);   // exact u - 8
            __nv_bfloat162 w2 = __hfma2(q2, s_hi, __hmul2(q2, s_lo));
            outw[i * 4 + pp] = *reinterpret_cast<uint32_t*>(&w2);
          }
        }
        // A tile of the stage in tensor memory: lane = row (this warp's quadrant), column = k / 2
        tmem_st16(tmem_d + ((uint32_t)((warp & 3) * 32) << 16) + kAccCols +
                      (uint32_t)(s * kATmemColsPerStage + h * 16), outw);
        tcgen05_fence_before();
        mbar_arrive(bar_deq(s));
      }
      if (!ok) *abort_flag = 1;
    }
    // epilogue: TMEM lane = output feature, column = token
    ok = __all_sync(0xffffffffu, ok);
    if (ok && __all_sync(0xffffffffu, mbar_wait(bar_acc, 0u, abort_flag))) {
      tcgen05_fence_after();
      const int quad = warp & 3;                          // TMEM lane quadrant this warp may read
      const int colhalf = (warp - kFirstDeqWarp) >> 2;    // 0 or 1
      const int n = n0 + quad * 32 + lane;
      const float bias = (p.bias != nullptr && n < p.N && blockIdx.z == 0) ? p.bias[n] : 0.0f;
      constexpr int kChunks = TOK / 16;
      for (int c = colhalf; c < kChunks; c += 2) {
        if (tok0 + c * 16 >= p.M) break;                  // warp-uniform
        uint32_t v[16];
        tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(c * 16), v);
        if (n < p.N) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = tok0 + c * 16 + j;
            if (t < p.M) {
              float acc = __uint_as_float(v[j]) + bias;
              if (OUT_MODE == kOutF32) {
                float* o = reinterpret_cast<float*>(p.out) + ((size_t)blockIdx.z * p.M + t) * p.ldo + n;
                *o = acc;
              } else {
                const size_t off = (size_t)t * p.ldo + n;
                if (p.residual) acc += __bfloat162float(p.residual[off]);
                reinterpret_cast<__nv_bfloat16*>(p.out)[off] = __float2bfloat16_rn(acc);
              }
            }
          }
        }
      }
    } else {
      ok = false;
      *abort_flag = 1;
    }
  }

  if (!ok && p.status != nullptr) atomicExch(p.status, 1);
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc(tmem_d, kTmemCols);
  }
}

// Sum of split-K partials in a fixed order, + bias + residual, to bf16.
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int splits, int M, int N,
                                     const float* __restrict__ bias, const __nv_bfloat16* __restrict__ residual,
                                     __nv_bfloat16* __restrict__ out, int ldo) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)M * N) return;
  const int t = (int)(idx / N), n = (int)(idx % N);
  float acc = 0.0f;
  for (int z = 0; z < splits; ++z) acc += part[((size_t)z * M + t) * N + n];
  if (bias) acc += bias[n];
  const size_t off = (size_t)t * ldo + n;
  if (residual) acc += __bfloat162float(residual[off]);
  out[off] = __float2bfloat16_rn(acc);
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// 2-D bf16 row-major [rows][cols] tensor map, box = 64 columns x box_rows rows, 128-byte swizzle.
int make_tmap_bf16(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return QZO_ERR_CUDA;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QZO_OK : QZO_ERR_CUDA;
}

int pick_tok_tile(int M) {
  if (M <= 16) return 16;
  if (M <= 32) return 32;
  if (M <= 64) return 64;
  if (M <= 128) return 128;
  return 256;
}

template <int TOK, bool DEQUANT, int OUT_MODE>
int launch_one(const CUtensorMap& tx, const CUtensorMap& tw, const GemmParams& p, dim3 grid, cudaStream_t st) {
  using Plan = SmemPlan<TOK, DEQUANT>;
  auto kern = w4a16_gemm_kernel<TOK, DEQUANT, OUT_MODE>;
  static bool configured = false;           // per instantiation
  if (!configured) {
    QZO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan::kDynamicBytes));
    configured = true;
  }
  QZO_LAUNCH(kern, grid, dim3(kThreads), Plan::kDynamicBytes, st, tx, tw, p);
  return QZO_OK;
}

template <bool DEQUANT, int OUT_MODE>
int launch_tok(int tok, const CUtensorMap& tx, const CUtensorMap& tw, const GemmParams& p, dim3 grid, cudaStream_t st) {
  switch (tok) {
    case 16: return launch_one<16, DEQUANT, OUT_MODE>(tx, tw, p, grid, st);
    case 32: return launch_one<32, DEQUANT, OUT_MODE>(tx, tw, p, grid, st);
    case 64: return launch_one<64, DEQUANT, OUT_MODE>(tx, tw, p, grid, st);
    case 128: return launch_one<128, DEQUANT, OUT_MODE>(tx, tw, p, grid, st);
    default: return launch_one<256, DEQUANT, OUT_MODE>(tx, tw, p, grid, st);
  }
}

}  // namespace

// Split-K plan: number of K slices for a problem (1 = none).  Slices hold an even number of
// k-blocks so that they start on a quantisation-group boundary.
int gemm_splits(int M, int K, int N) {
  const int tok = pick_tok_tile(M);
  const int tiles = ceil_div(N, kTileN) * ceil_div(M, tok);
  const int groups = ceil_div(K, kGroup);
  if (tiles >= 120 || groups < 8) return 1;
  int splits = 296 / tiles;                      // aim at two CTAs per SM
  if (splits > groups / 4) splits = groups / 4;  // at least four groups per slice
  if (splits > 16) splits = 16;
  return splits < 1 ? 1 : splits;
}

size_t gemm_workspace_bytes(int M, int K, int N) {
  const int splits = gemm_splits(M, K, N);
  if (splits <= 1) return 0;
  return (size_t)splits * M * N * sizeof(float);
}

// Y = X W' (+ bias) (+ residual) with W' de-quantised from int4 and perturbed scales.
int launch_perturbed_gemm(const __nv_bfloat16* d_x, const void* d_wq, const __nv_bfloat16* d_scales,
                          const float* d_bias, const __nv_bfloat16* d_residual, __nv_bfloat16* d_y, int ldo,
                          int M, int K, int N, uint64_t seed, uint64_t idx_base, int sign, float eps,
                          void* d_ws, size_t ws_bytes, int* d_status, cudaStream_t st) {
  if (M <= 0 || K <= 0 || N <= 0 || (K % 8) != 0 || (N % 8) != 0 || (idx_base % 4) != 0) return QZO_ERR_BAD_ARG;
  const int tok = pick_tok_tile(M);
  CUtensorMap tx;
  QZO_TRY(make_tmap_bf16(&tx, d_x, M, K, tok));
  const int splits = gemm_splits(M, K, N);
  GemmParams p{};
  p.wq = reinterpret_cast<const uint8_t*>(d_wq);
  p.scales = d_scales;
  p.M = M; p.K = K; p.N = N;
  p.num_kb = ceil_div(K, kBlockK);
  p.seed = seed; p.idx_base = idx_base;
  p.sign_eps = (float)sign * eps;
  p.status = d_status;
  const int groups = ceil_div(K, kGroup);
  if (splits <= 1) {
    p.bias = d_bias; p.residual = d_residual; p.out = d_y; p.ldo = ldo;
    p.kb_per_split = ceil_div(p.num_kb, 2) * 2;
    dim3 grid(ceil_div(N, kTileN), ceil_div(M, tok), 1);
    return launch_tok<true, kOutBf16>(tok, tx, tx, p, grid, st);
  }
  const size_t need = (size_t)splits * M * N * sizeof(float);
  if (d_ws == nullptr || ws_bytes < need) return QZO_ERR_WORKSPACE;
  const int groups_per = ceil_div(groups, splits);
  const int zdim = ceil_div(groups, groups_per);           // every slice is non-empty
  p.bias = nullptr; p.residual = nullptr; p.out = d_ws; p.ldo = N;
  p.kb_per_split = groups_per * 2;
  dim3 grid(ceil_div(N, kTileN), ceil_div(M, tok), zdim);
  QZO_TRY((launch_tok<true, kOutF32>(tok, tx, tx, p, grid, st)));
  const int64_t total = (int64_t)M * N;
  QZO_LAUNCH(splitk_reduce_kernel, dim3((unsigned)ceil_div64(total, 256)), dim3(256), 0, st,
             reinterpret_cast<const float*>(d_ws), zdim, M, N, d_bias, d_residual, d_y, ldo);
  return QZO_OK;
}

// logits[t][v] = sum_k X[t][k] Wh[v][k]: bf16 weights [V][K] row-major, fp32 output [M][V].
int launch_bf16_gemm_f32out(const __nv_bfloat16* d_x, const __nv_bfloat16* d_w, float* d_out, int M, int K, int N,
                            int* d_status, cudaStream_t st) {
  if (M <= 0 || K <= 0 || N <= 0 || (K % 8) != 0) return QZO_ERR_BAD_ARG;
  const int tok = pick_tok_tile(M);
  CUtensorMap tx, tw;
  QZO_TRY(make_tmap_bf16(&tx, d_x, M, K, tok));
  QZO_TRY(make_tmap_bf16(&tw, d_w, N, K, kTileN));
  GemmParams p{};
  p.M = M; p.K = K; p.N = N; p.ldo = N;
  p.out = d_out;
  p.num_kb = ceil_div(K, kBlockK);
  p.kb_per_split = ceil_div(p.num_kb, 2) * 2;
  p.status = d_status;
  dim3 grid(ceil_div(N, kTileN), ceil_div(M, tok), 1);
  return launch_tok<false, kOutF32>(tok, tx, tw, p, grid, st);
}

}  // namespace qzo
