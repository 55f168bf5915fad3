// Perturbed W4A16 GEMM for sm_100a: Y[t][n] = sum_k X[t][k] (s[k/128][n] + sign eps z_i) q[k][n].
//
// Eq. 4 (w = Delta * w_bar) is evaluated in the kernel's prologue with the perturbed scale
// of Eq. 5, Delta' = Delta + sign eps z, formed in fp32 from the stored bf16 scale and a
// Gaussian z regenerated from (seed, logical scale index); the stored scales are never
// written.  The contraction runs on the tcgen05 tensor cores with the accumulator in TMEM.
//
// Tile roles.  The de-quantised weight tile is the MMA's A operand (UMMA M = 128 output
// features) and lives in tensor memory; the activation tile is the B operand (UMMA N = TOK
// tokens, 16..256) in shared memory, so that one de-quantised weight feeds TOK multiply-adds
// and small token counts do not waste tensor rows.  D[n][t] sits in TMEM with lane = output
// feature, column = token.
//
// The kernel is persistent: one CTA per SM walks a static list of work units (a 128-feature x
// TOK-token tile of one linear, optionally one K slice of it).  Up to three linears that share
// the activations (q, k, v or gate, up) are served by one launch; the logical scale index of a
// scale never depends on that grouping.
//
// Warp roles (25 warps; 29 at token tiles up to 128):
//   warp 0       TMA producer of the B ring: activation tiles (2-D tensor map, 128-byte swizzle)
//   warp 1       MMA issuer (one elected lane), owns the TMEM allocation; token tiles up to 128: eight MMAs and
//                one commit per quantisation group (the commit frees the group's slot in both rings)
//   warp 2       producer of the A ring: packed int4 tiles (one 8 KiB bulk copy per quantisation group)
//   warp 3       watch warp: does the mbarrier waits the issuer depends on and publishes a count; token tiles up
//                to 128: its lanes test the barriers of the next groups at once and it publishes in batches
//   warps 4-7    scale warps: Philox4x32-10 + Box-Muller, s' = s + sign eps z in fp32, split
//                into bf16 hi + lo parts, written next to the nibbles of the group's A slot
//   warps 8-15   de-quantisers: nibbles -> bf16 (u - 8) * s' written to the A stages in TMEM; teams of four
//    (8-19)      warps take the quantisation groups in turn: two teams at 256-token tiles, three below
//   next 8       epilogue: TMEM -> registers (+ bias) -> bf16 rows in shared memory, 32 tokens per pass
//                (the last passes of a full tile wait in registers: the accumulator is released first)
//   last warp    store warp: issues the TMA store of every staged pass (three staging buffers), so
//                that the warps draining the single accumulator never wait for a store to be issued
// Every wait on an mbarrier is bounded; when a wait expires the CTA records an error in
// the status word, drains its copies and leaves through the common exit (TMEM is freed).
#include "qzo_common.cuh"
#include "philox.cuh"
#include "launch.cuh"
#include "layers.cuh"

#include <cuda.h>
#include <cstring>
#include <mutex>

namespace qzo {

namespace {

constexpr int kATmemColsPerStage = kBlockK / 2;   // 64 bf16 along K = 32 TMEM columns of 32 bits
constexpr int kMaxASlots = 7;         // A-ring slots (quantisation groups in flight); each holds its perturbed scales
constexpr int kNumScaleWarps = 4;
constexpr int kNumEpiWarps = 8;
constexpr int kAProducerWarp = 2;
constexpr int kWatchWarp = 3;          // waits on the mbarriers on behalf of the MMA issuer
constexpr int kFirstScaleWarp = 4;
constexpr int kFirstDeqWarp = kFirstScaleWarp + kNumScaleWarps;
// De-quantiser teams of four warps (one warp per tensor-memory lane quadrant), taking quantisation groups in turn:
// two at 256-token tiles (72 registers per thread there; a third team would not fit the register file) and
// for bf16 weights (where they idle), three at token tiles up to 128, where every role gets an issue slot only now
// and then and a third team shortens the de-quantisers' turn-around.  The warps after them follow.
template <int TOK, int WMODE>
struct Roles {
  static constexpr int kDeqTeams = (WMODE != 0 && TOK <= 128) ? 3 : 2;
  static constexpr int kNumDeqWarps = 4 * kDeqTeams;
  static constexpr int kFirstEpiWarp = kFirstDeqWarp + kNumDeqWarps;
  static constexpr int kStoreWarp = kFirstEpiWarp + kNumEpiWarps;   // issues the TMA stores of the finished tiles
  static constexpr int kNumWarps = kStoreWarp + 1;
  static constexpr int kThreads = kNumWarps * 32;
};
constexpr long long kWaitLimitCycles = 4000000000LL;   // ~2 s at boost clock
constexpr int kSmemBudget = 227 * 1024;

constexpr int kWTileBytes = kTileN * kBlockK * 2;      // 16 KiB bf16 A tile (bf16-weight path)
constexpr int kCookedScaleBytes = kTileN * 8;          // {hi,hi},{lo,lo} per output feature
constexpr int kRawScaleBytes = kTileN * 2;             // one row of stored bf16 scales of the tile's features
constexpr int kLutSmemBytes = 16 * 32 * 4;             // table mode: every codebook value as a bf16 pair, one copy per lane (bank)

// How the A operand comes about.
enum WeightMode {
  kWBf16 = 0,     // bf16 [N][K] matrix loaded as it is (lm_head)
  kWInt4 = 1,     // packed int4, one scale per group of 128 k: w = (u - 8) s'   (Eq. 4, the paper's GPTQ setting)
  kWTable16 = 2   // packed 4-bit codes into a 16-entry table, one scale per block of 64 k: w = table[u] s'
                  // (block-scaled codebook storage such as NF4; only the prologue differs)
};

enum OutMode { kOutBf16 = 0, kOutF32 = 1 };

struct LinearDesc {
  const uint8_t* wq;              // kernel-layout int4 (dequant mode)
  const __nv_bfloat16* scales;    // [G][N] of this linear
  const float* bias;              // [N] or null
  void* out;                      // bf16 [M][ldo]  or  float [splits][M][ldo]
  unsigned long long idx_base;    // logical index of scale [0][0]
  int N, ldo;
  int n_tiles;                    // ceil(N / 128)
};

struct GemmParams {
  LinearDesc lin[kMaxGroupedLinears];
  int n_lin, tiles_n_total;
  int M, K;
  int num_kb;                     // ceil(K / 64)
  int kb_per_split;               // even number of k-blocks per K slice
  int splits, m_tiles, total_units;
  unsigned long long seed;
  float sign_eps;                 // sign * eps (0 when unperturbed); with `sp`: the sign alone
  const StepParams* sp;           // non-null: seed and eps are read from here (a recorded step)
  int pair_rows;                  // > 0: token rows from this one on take -sign_eps (both passes of a step in one launch)
  int* status;
  long long wait_limit;           // cycles after which a device-side wait gives up
  int scale_row_mul;              // 1: one row of scales per group / block of k; 0: one row for all k (channel-wise scales)
  int skip_group;                 // >= 0 (tests only): the A producer announces this group's copies but does not issue them
  float lut[16];                  // table mode: the 16 codebook values (a nibble is an index into them)
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
// One test of the barrier that never suspends the thread (try_wait may park it for a while when the phase
// is not complete): for a warp whose lanes look at several barriers, most of them not due yet.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Up to 1024 polls of the barrier in a short loop; true when the phase completed.
__device__ __forceinline__ bool mbar_poll(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .u32 n;\n\t"
      "mov.u32 n, 1024;\n"
      "POLL:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "@p bra.uni DONE;\n\t"
      "sub.u32 n, n, 1;\n\t"
      "setp.ne.u32 p, n, 0;\n\t"
      "@p bra.uni POLL;\n\t"
      "mov.u32 %0, 0;\n\t"
      "bra.uni END;\n"
      "DONE:\n\t"
      "mov.u32 %0, 1;\n"
      "END:\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// Bounded wait: false when the limit expired or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
  if (mbar_poll(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_poll(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) return false;
  }
}
// Same bound, for waits that are long and not latency-critical: sleeps between polls so that the
// waiting warp leaves the issue slots to the working ones.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    __nanosleep(256);
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 0x3F) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) return false;
    }
  }
}
// Hardware barrier among `nthreads` threads of the CTA (whole warps): the waiting warps are parked,
// they do not poll.  Every participating warp reaches every such barrier, also after a failed wait.
__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// Signs a hardware barrier without waiting for it (producer side of a producer / consumer pair).
__device__ __forceinline__ void named_bar_arrive(uint32_t id, uint32_t nthreads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
      ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until at most N of this thread's most recent bulk-copy groups still read their source.
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_group0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}
// One lane of the (converged) warp; the surrounding code stays warp-uniform, so that loop state
// and descriptors live in uniform registers.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ int ld_acquire_shared(uint32_t addr) {
  int v;
  asm volatile("ld.acquire.cta.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_shared(uint32_t addr, int v) {
  asm volatile("st.release.cta.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
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
// The four MMAs of one 64-deep k-block (K = 16 each) with A in tensor memory, in one instruction
// sequence: A advances by 8 TMEM columns, the B descriptor by 32 bytes (2 in its address field) per
// step; only the first may overwrite the accumulator.
__device__ __forceinline__ void umma_bf16_tmem_a_x4(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                                    uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p, t;\n\t.reg .b32 a1, a2, a3;\n\t.reg .b64 b1, b2, b3;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.eq.b32 t, 0, 0;\n\t"
      "add.u32 a1, %1, 8;\n\t add.u32 a2, %1, 16;\n\t add.u32 a3, %1, 24;\n\t"
      "add.u64 b1, %2, 2;\n\t add.u64 b2, %2, 4;\n\t add.u64 b3, %2, 6;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a1], b1, %3, t;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a2], b2, %3, t;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a3], b3, %3, t;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate_first)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t v[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
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
constexpr int cmin(int a, int b) { return a < b ? a : b; }

// Two rings feed the MMA.  The A ring (packed nibbles in shared memory -> de-quantised bf16 in
// tensor memory) is deep and cheap, so the de-quantisers run well ahead of the tensor pipe; the
// B ring holds the activation tiles.  A finished bf16 tile leaves in passes of up to 32 tokens
// through three staging buffers, each pass as one TMA store.
template <int TOK, int WMODE, int OUT_MODE>
struct SmemPlan {
  static constexpr bool DEQUANT = WMODE != kWBf16;
  static constexpr bool LUT = WMODE == kWTable16;
  static constexpr int kScaleRows = LUT ? 2 : 1;       // rows of scales per ring slot (a slot is 128 k)
  // one slot of the nibble ring: a group's packed nibbles, its perturbed scales, its stored scales
  static constexpr int kOffCookedInSlot = 2 * kPackedTileBytes;
  static constexpr int kOffRawInSlot = kOffCookedInSlot + kScaleRows * kCookedScaleBytes;
  static constexpr int kNibSlotBytes = kOffRawInSlot + kScaleRows * kRawScaleBytes;
  static constexpr int kAccCols = TOK < 32 ? 32 : TOK;
  static constexpr int kXTileBytes = TOK * kBlockK * 2;
  // int4 path: A stage = 4 KiB of packed nibbles; bf16 path: A stage = 16 KiB bf16 tile (read by the MMA)
  static constexpr int kAStageBytes = DEQUANT ? kPackedTileBytes : kWTileBytes;
  static constexpr int kPassTok = TOK < 32 ? TOK : 32;
  static constexpr int kPasses = TOK / kPassTok;
  static constexpr int kStagingBufBytes = kPassTok * kTileN * 2;
  // three staging buffers: a pass waits for the TMA store issued two passes earlier, not for the last one
  static constexpr int kStagingBufs = 3;
  static constexpr int kStagingBytes = OUT_MODE == kOutBf16 ? kStagingBufs * kStagingBufBytes : 0;
  static constexpr int kFixedBytes = kStagingBytes + 1024 + 1024 + (LUT ? kLutSmemBytes : 0);
  // int4 path: the A ring (4 KiB of nibbles + 32 TMEM columns per stage) is as deep as tensor memory
  // allows, the B ring takes the shared memory that is left; bf16 path: both rings alike
  static constexpr int kStagesTmem = (512 - kAccCols) / kATmemColsPerStage;
  // A slot of the int4 path = one quantisation group = two k-blocks: one 8 KiB bulk copy, one wait
  // and one arrival per group for the producer, the de-quantisers and the MMA warp
  static constexpr int kAGroup = DEQUANT ? 2 : 1;                  // k-blocks per A-ring slot
  static constexpr int kAStages = DEQUANT ? cmin(2 * kMaxASlots, kStagesTmem) / 2 * 2 : 4;
  static constexpr int kASlots = kAStages / kAGroup;
  // Token tiles up to 128: the B ring also works in slots of two k-blocks (one wait, one expect and one
  // commit per quantisation group); there the per-k-block cost of the single-thread roles is the limit
  static constexpr int kBGroup = (DEQUANT && TOK <= 128) ? 2 : 1;
  // bytes of one slot of the ring that the A producer fills: int4 path: nibbles and scales of a group (the
  // de-quantised operand lives in tensor memory); bf16 path: the 16 KiB tile the MMA reads
  static constexpr int kNibBytes = DEQUANT ? kNibSlotBytes : kAStageBytes;
  // up to 8 stages; 16 where a stage is at most 4 KiB (token tiles up to 32): there a slot's round trip (its
  // group's MMAs retire, the producer sees it, the tile arrives from L2) is longer than four groups last
  static constexpr int kBStagesMax = (DEQUANT && TOK <= 32) ? 16 : 8;
  static constexpr int kBStages = DEQUANT ? cmin(kBStagesMax, (kSmemBudget - kFixedBytes - kASlots * kNibBytes) / kXTileBytes) / kBGroup * kBGroup : 4;
  static constexpr int kBSlots = kBStages / kBGroup;
  static_assert(kBSlots >= 2 && kASlots >= 2, "pipelines need at least two stages");
  // int4 path: the nibble ring is deeper than the tensor-memory stages wherever shared memory is left (small
  // token tiles): its slots are released as soon as the de-quantisers have read them, so the copies in
  // flight, not the de-quantise / MMA / commit round of a tensor-memory stage, cover the HBM latency
  static constexpr int kNibCap = TOK <= 64 ? 16 : 8;
  // Token tiles up to 128: the stored scales of a group travel with its nibbles (a second bulk copy into the
  // slot), so that the scale warps never wait for a load from HBM.  256-token tiles keep the scale warps'
  // own early load: there the ring has four slots, and the perturbed scales must be written the moment a
  // slot is released.
  static constexpr bool kRawViaCopy = DEQUANT && TOK <= 128;
  static constexpr int kNibLeft = (kSmemBudget - kFixedBytes - kBStages * kXTileBytes - 3 * 8 * 16 - 64) / kNibBytes;
  static constexpr int kNibSlots = DEQUANT ? (kNibLeft < kASlots ? kASlots : cmin(kNibCap, kNibLeft)) : kASlots;
  static_assert(kNibSlots >= kASlots, "nibble ring at least as deep as the tensor-memory stages");
  static constexpr int kOffB = 0;
  static constexpr int kOffA = kBStages * kXTileBytes;                 // nibble ring / bf16 A ring
  static constexpr int kOffStaging = kOffA + kNibSlots * kNibBytes;
  static constexpr int kOffLut = kOffStaging + kStagingBytes;
  static constexpr int kOffBars = kOffLut + (LUT ? kLutSmemBytes : 0);
  static constexpr int kNumBars = 2 * kBStages + 3 * kNibSlots + 2 * kAStages + 2;
  static constexpr int kOffMisc = kOffBars + kNumBars * 8;
  static constexpr int kTotal = kOffMisc + 32;
  static constexpr int kDynamicBytes = kTotal + 1024;      // slack for the 1024-byte alignment
  static_assert(kDynamicBytes <= kSmemBudget, "shared memory budget");
  static constexpr uint32_t kUsedCols = DEQUANT ? kAccCols + kAStages * kATmemColsPerStage : kAccCols;
  static constexpr uint32_t kTmemCols = kUsedCols <= 32 ? 32 : kUsedCols <= 64 ? 64 : kUsedCols <= 128 ? 128
                                        : kUsedCols <= 256 ? 256 : 512;
  static_assert(kUsedCols <= 512, "TMEM budget");
};

struct Unit {
  int lin, n0, tok0, z, kb_begin, nkb;
};
// Work unit u of the launch: K slice z, token tile, then the feature tiles of every linear.
// Consecutive units (which run at the same time on different SMs) share the activation tile.
__device__ __forceinline__ Unit decode_unit(const GemmParams& p, int u, int tok_tile) {
  Unit w;
  const int per = p.tiles_n_total * p.m_tiles;
  w.z = u / per;
  const int r = u - w.z * per;
  const int m = r / p.tiles_n_total;
  int nn = r - m * p.tiles_n_total;
  int lin = 0;
  while (lin + 1 < p.n_lin && nn >= p.lin[lin].n_tiles) { nn -= p.lin[lin].n_tiles; ++lin; }
  w.lin = lin;
  w.n0 = nn * kTileN;
  w.tok0 = m * tok_tile;
  w.kb_begin = w.z * p.kb_per_split;
  w.nkb = min(w.kb_begin + p.kb_per_split, p.num_kb) - w.kb_begin;      // >= 1 by construction of the grid
  return w;
}

// Ring position: stage index and the parity of the round it is in.
struct Ring {
  int s = 0;
  uint32_t ph = 0;
  __device__ __forceinline__ void next(int stages) {
    if (++s == stages) { s = 0; ph ^= 1u; }
  }
};

// ----------------------------------------------------------------------------- the kernel
// WMODE (WeightMode): kWInt4 / kWTable16: A operand produced from packed 4-bit codes + perturbed scales;
// kWBf16: A operand is a bf16 [N][K] row-major matrix loaded through tmap_w (lm_head).
template <int TOK, int WMODE, int OUT_MODE>
__global__ void __launch_bounds__((Roles<TOK, WMODE>::kThreads), 1)
w4a16_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                  const __grid_constant__ CUtensorMap tmap_y0, const __grid_constant__ CUtensorMap tmap_y1,
                  const __grid_constant__ CUtensorMap tmap_y2, const __grid_constant__ GemmParams p) {
  using Plan = SmemPlan<TOK, WMODE, OUT_MODE>;
  using R = Roles<TOK, WMODE>;
  constexpr int kDeqTeams = R::kDeqTeams;
  constexpr int kFirstEpiWarp = R::kFirstEpiWarp;
  constexpr int kStoreWarp = R::kStoreWarp;
  constexpr bool DEQUANT = Plan::DEQUANT;
  constexpr bool LUT = Plan::LUT;
  constexpr int kScaleRows = Plan::kScaleRows;
  constexpr int kAStages = Plan::kAStages;
  constexpr int kASlots = Plan::kASlots;
  constexpr int kAGroup = Plan::kAGroup;
  constexpr int kBStages = Plan::kBStages;
  constexpr int kBSlots = Plan::kBSlots;
  constexpr int kBGroup = Plan::kBGroup;
  // Token tiles up to 128: a slot of either ring is one quantisation group, and both are free when the group's
  // MMAs have retired, so the issuer signs ONE barrier per group (a tcgen05.commit costs the issuing thread
  // about as much as four MMAs): the tensor-memory slot's "empty" barrier, which the B producer watches too.
  constexpr bool kMergedRelease = DEQUANT && kAGroup == 2 && kBGroup == 2;
  constexpr uint32_t kAccCols = Plan::kAccCols;
  constexpr uint32_t kTmemCols = Plan::kTmemCols;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const smem = smem_raw + (base - smem_u32(smem_raw));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const long long wait_limit = p.wait_limit;      // bound of every wait, in cycles (about two seconds outside tests)

  const uint32_t bar0 = base + Plan::kOffBars;
  auto bar_b_full = [&](int s) { return bar0 + 8u * s; };                        // activation tile landed
  auto bar_b_empty = [&](int s) { return bar0 + 8u * (kBStages + s); };          // MMAs that read it retired
  constexpr int kNibSlots = Plan::kNibSlots;
  // nibble ring (int4 path) / A ring (bf16 path): full = nibbles landed and perturbed scales written (bf16
  // path: unused, the B barrier counts both tiles); raw = the group's stored scales landed; free = the
  // de-quantisers have read the slot (bf16 path: the MMAs that read it retired)
  auto bar_nib_full = [&](int s) { return bar0 + 8u * (2 * kBStages + s); };
  auto bar_nib_raw = [&](int s) { return bar0 + 8u * (2 * kBStages + kNibSlots + s); };
  auto bar_nib_free = [&](int s) { return bar0 + 8u * (2 * kBStages + 2 * kNibSlots + s); };
  // tensor-memory stages of the de-quantised operand (one slot = one group = two k-blocks)
  auto bar_a_deq = [&](int s) { return bar0 + 8u * (2 * kBStages + 3 * kNibSlots + s); };                // de-quantised
  auto bar_a_empty = [&](int s) { return bar0 + 8u * (2 * kBStages + 3 * kNibSlots + kAStages + s); };   // MMAs that read it retired
  const uint32_t bar_acc_full = bar0 + 8u * (2 * kBStages + 3 * kNibSlots + 2 * kAStages);   // accumulator complete
  const uint32_t bar_acc_empty = bar_acc_full + 8u;                              // accumulator drained
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(smem + Plan::kOffMisc);
  uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(smem + Plan::kOffMisc + 4);
  volatile int* const never_set = reinterpret_cast<volatile int*>(smem + Plan::kOffMisc + 8);   // stays 0
  // The epilogue warps parked on a hardware barrier learn from this whether their polling warp gave
  // up: it holds the first unit count that must not be started.  Written by that warp only, before it
  // reaches the barrier, so that every warp leaves the loop at the same barrier.
  volatile int* const epi_stop = reinterpret_cast<volatile int*>(smem + Plan::kOffMisc + 12);
  // Number of k-blocks (of this CTA, all units) whose operands the watch warp has seen ready; -1 when it
  // gave up.  The MMA issuer reads this word instead of polling mbarriers: a ready mbarrier wait costs
  // the issuing thread about three times as much as a shared-memory load, and that thread is the
  // bottleneck of the kernel.
  const uint32_t ready_addr = base + Plan::kOffMisc + 16;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    *never_set = 0;
    *epi_stop = 0x7fffffff;
    *reinterpret_cast<volatile int*>(smem + Plan::kOffMisc + 16) = 0;
    for (int s = 0; s < kBSlots; ++s) {
      // bf16 path: one barrier tells the MMA warp that both tiles of a stage have landed (rings of
      // equal depth).  int4 path: the A ring is deeper than the B ring, so the de-quantisers signal
      // their own barrier (an arrival on the B barrier could fall into its previous phase)
      mbar_init(bar_b_full(s), DEQUANT ? 1 : 2);
      mbar_init(bar_b_empty(s), 1);
    }
    for (int s = 0; s < kNibSlots; ++s) {
      // int4 path: the slot is full when its nibbles have landed AND its perturbed scales are written
      mbar_init(bar_nib_full(s), DEQUANT ? 2 : 1);
      mbar_init(bar_nib_raw(s), 1);
      mbar_init(bar_nib_free(s), DEQUANT ? 4 : 1);   // one team of four de-quantiser warps per group
    }
    for (int s = 0; s < kASlots; ++s) {
      mbar_init(bar_a_deq(s), 4);
      mbar_init(bar_a_empty(s), 1);
    }
    mbar_init(bar_acc_full, 1);
    mbar_init(bar_acc_empty, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (LUT && threadIdx.x < 512) {
    // codebook value e as a bf16 pair {t, t}, one copy per lane: entry (e, lane) sits in bank `lane`
    const uint32_t t16 = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(p.lut[threadIdx.x >> 5]));
    reinterpret_cast<uint32_t*>(smem + Plan::kOffLut)[threadIdx.x] = t16 | (t16 << 16);
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  bool ok = true;
  // threads at the epilogue's hardware barriers: for bf16 tiles the store warp takes part
  constexpr int kEpiBarThreads = (kNumEpiWarps + (OUT_MODE == kOutBf16 ? 1 : 0)) * 32;
  constexpr uint32_t kBarUnit = 1, kBarStaged = 2, kBarFree = 3, kBarDrained = 4;

  if (warp == 0 || warp == kAProducerWarp) {
    // ------------------------------------------------------------------ TMA producers
    // warp 0 feeds the B ring (activation tiles), warp 2 the A ring (packed nibbles / bf16 weights)
    if (lane == 0) {
      const bool is_b = warp == 0;
      const int stages = is_b ? kBSlots : kNibSlots;
      Ring ring;
      int issued = 0;
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u, TOK);
        const LinearDesc& L = p.lin[w.lin];
        if (is_b) {
          for (int it = 0; it < w.nkb; it += kBGroup) {
            const int nk = min(kBGroup, w.nkb - it);          // k-blocks of this slot
            if (kMergedRelease) {
              // the slot's previous group (kBSlots groups back) is released by that group's tensor-memory
              // slot: one commit of the issuer frees both
              const int x = issued - kBSlots;
              if (x >= 0 && !mbar_wait(bar_a_empty(x % kASlots), (uint32_t)(x / kASlots) & 1u, abort_flag, wait_limit)) {
                ok = false;
                break;
              }
            } else if (!mbar_wait(bar_b_empty(ring.s), ring.ph ^ 1u, abort_flag, wait_limit)) {
              ok = false;
              break;
            }
            mbar_arrive_expect_tx(bar_b_full(ring.s), (uint32_t)(nk * Plan::kXTileBytes));
            for (int j = 0; j < nk; ++j)
              tma_load_2d(base + Plan::kOffB + (ring.s * kBGroup + j) * Plan::kXTileBytes, &tmap_x, bar_b_full(ring.s),
                          (w.kb_begin + it + j) * kBlockK, w.tok0);
            ring.next(stages);
            ++issued;
          }
        } else {
          for (int it = 0; it < w.nkb; it += kAGroup) {
            const int kb = w.kb_begin + it;
            const int nk = min(kAGroup, w.nkb - it);         // k-blocks of this slot (the last group of an odd K has one)
            if (!mbar_wait(bar_nib_free(ring.s), ring.ph ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
            const uint32_t dst = base + Plan::kOffA + ring.s * Plan::kNibBytes;
            if (DEQUANT) {
              // tests of the bounded waits: one group's copies are announced and never issued, so every wait
              // that depends on them runs out
              const bool skip = issued == p.skip_group;
              mbar_arrive_expect_tx(bar_nib_full(ring.s), (uint32_t)(nk * kPackedTileBytes));
              if (!skip)
                bulk_load(dst, L.wq + ((size_t)(w.n0 / kTileN) * p.num_kb + kb) * kPackedTileBytes,
                          (uint32_t)(nk * kPackedTileBytes), bar_nib_full(ring.s));
              // the group's stored scales of this tile's features travel with the nibbles (N is a multiple of 8
              // and the scale rows are 16-byte aligned, so is every run of them)
              if (Plan::kRawViaCopy) {
                const uint32_t raw_bytes = (uint32_t)min(kTileN, L.N - w.n0) * 2u;
                // int4: the group's row of scales; table mode: one row per k-block of the slot
                const int rows = LUT ? nk : 1;
                const int row0 = LUT ? kb : (kb >> 1);
                mbar_arrive_expect_tx(bar_nib_raw(ring.s), raw_bytes * (uint32_t)rows);
                for (int j = 0; j < rows && !skip; ++j)
                  bulk_load(dst + Plan::kOffRawInSlot + j * kRawScaleBytes, L.scales + (size_t)((row0 + j) * p.scale_row_mul) * L.N + w.n0, raw_bytes,
                            bar_nib_raw(ring.s));
              }
            } else {
              mbar_arrive_expect_tx(bar_b_full(ring.s), Plan::kAStageBytes);
              tma_load_2d(dst, &tmap_w, bar_b_full(ring.s), kb * kBlockK, w.n0);
            }
            ring.next(stages);
            ++issued;
          }
        }
      }
      if (!ok) {
        // drain: give the copies already issued a bounded chance to land before the CTA exits
        *abort_flag = 1;
        const int pending = min(issued, stages);
        for (int j = 0; j < pending; ++j) {
          const int idx = issued - 1 - j;
          // int4 path: the slot's "full" barrier also counts a scale warp, which may have given up; its copies
          // are waited for through the stored scales' barrier (issued last) where there is one
          const uint32_t bar = (is_b || !DEQUANT) ? bar_b_full(idx % stages)
                                                  : (Plan::kRawViaCopy ? bar_nib_raw(idx % stages) : bar_nib_full(idx % stages));
          mbar_wait(bar, (uint32_t)(idx / stages) & 1u, never_set, wait_limit);
        }
        // a nibble copy issued just before an awaited scale copy may land a moment after it
        if (!is_b && Plan::kRawViaCopy) __nanosleep(50000);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop (warp-uniform control flow and addresses); one elected lane
    // issues the MMAs and the commits.
    constexpr uint32_t idesc = umma_idesc_bf16(kTileN, TOK);
    const bool leader = elect_one();
    const uint64_t bdesc0 = umma_desc_k_major_sw128(base + Plan::kOffB);   // stage s: start address + s * tile bytes
    Ring ra, rb;
    int itg = 0;
    int seen = 0;                                             // k-blocks the watch warp had published at the last look
    // Token tiles up to 128: one pass of the loop per quantisation group (its two k-blocks sit side by side in both
    // rings): eight MMAs and one commit with as little around them as possible.  This thread's instruction stream
    // is what the small-token GEMM waits for (it shares its scheduler with the de-quantisers).
    for (int u = blockIdx.x; kMergedRelease && u < p.total_units && ok; u += gridDim.x) {
      const Unit w = decode_unit(p, u, TOK);
      const int ngroups = (w.nkb + 1) >> 1;
      for (int g = 0; g < ngroups; ++g) {
        const int nk = (2 * g + 1 < w.nkb) ? 2 : 1;
        if (seen < itg + nk) {
          seen = ld_acquire_shared(ready_addr);
          if (seen >= 0 && seen < itg + nk) {
            const long long t0 = clock64();
            do {
              seen = ld_acquire_shared(ready_addr);
            } while (seen >= 0 && seen < itg + nk && clock64() - t0 < wait_limit);
          }
          if (seen < itg + nk) { ok = false; break; }         // the watch warp gave up (-1), or the limit expired
          tcgen05_fence_after();
        }
        if (leader) {
          const uint32_t a_tmem = tmem_d + kAccCols + (uint32_t)(ra.s * kAGroup * kATmemColsPerStage);
          const uint64_t bdesc = bdesc0 + (uint64_t)(rb.s * kBGroup * (Plan::kXTileBytes >> 4));
          umma_bf16_tmem_a_x4(tmem_d, a_tmem, bdesc, idesc, g > 0 ? 1u : 0u);
          if (nk == 2) umma_bf16_tmem_a_x4(tmem_d, a_tmem + kATmemColsPerStage, bdesc + (uint64_t)(Plan::kXTileBytes >> 4), idesc, 1u);
          umma_commit(bar_a_empty(ra.s));                     // frees the group's slot in both rings
        }
        itg += nk;
        ra.next(kASlots);
        rb.next(kBSlots);
      }
      if (!ok) break;
      if (leader) umma_commit(bar_acc_full);
      __syncwarp();
    }
    for (int u = blockIdx.x; !kMergedRelease && u < p.total_units && ok; u += gridDim.x) {
      const Unit w = decode_unit(p, u, TOK);
      for (int it = 0; it < w.nkb; ++it, ++itg) {
        const int j = it % kAGroup;                           // position inside the A slot
        if (seen <= itg) {
          // wait (bounded) until the watch warp has seen this k-block's operands ready and, for the
          // first k-block of a unit, the accumulator drained.  The count it publishes often covers several
          // k-blocks: the issuer asks again only when it has used up what it last saw.
          seen = ld_acquire_shared(ready_addr);
          if (seen >= 0 && seen <= itg) {
            const long long t0 = clock64();
            do {
              seen = ld_acquire_shared(ready_addr);
            } while (seen >= 0 && seen <= itg && clock64() - t0 < wait_limit);
          }
          if (seen <= itg) { ok = false; break; }             // the watch warp gave up (-1), or the limit expired
          tcgen05_fence_after();
        }
        const bool slot_done = j == kAGroup - 1 || it == w.nkb - 1;
        const int jb = it % kBGroup;                          // position inside the B slot
        const bool bslot_done = jb == kBGroup - 1 || it == w.nkb - 1;
        const uint64_t bdesc = bdesc0 + (uint64_t)((rb.s * kBGroup + jb) * (Plan::kXTileBytes >> 4));
        if (leader) {
          if (DEQUANT) {
            const uint32_t a_tmem = tmem_d + kAccCols + (uint32_t)((ra.s * kAGroup + j) * kATmemColsPerStage);
            static_assert(kBlockK == 64, "four K = 16 steps per k-block");
            umma_bf16_tmem_a_x4(tmem_d, a_tmem, bdesc, idesc, it > 0 ? 1u : 0u);
          } else {
            const uint64_t adesc = umma_desc_k_major_sw128(base + Plan::kOffA + ra.s * Plan::kNibBytes);
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)
              umma_bf16(tmem_d, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                        (it > 0 || k > 0) ? 1u : 0u);
          }
          if (bslot_done && !kMergedRelease) umma_commit(bar_b_empty(rb.s)); // releases the B slot
          if (slot_done) umma_commit(DEQUANT ? bar_a_empty(ra.s) : bar_nib_free(ra.s));  // and, after its last k-block, the A slot
        }
        if (slot_done) ra.next(kASlots);
        if (bslot_done) rb.next(kBSlots);
      }
      if (ok && leader) umma_commit(bar_acc_full);
      __syncwarp();
    }
    if (!ok) *abort_flag = 1;
  } else if (warp == kWatchWarp) {
    // ------------------------------------------------------------------ watch warp
    // Performs the (bounded) mbarrier waits the MMA issuer depends on, ahead of it in time, and publishes
    // the count of ready k-blocks.
    Ring ra, rb;
    int useq = 0, itg = 0;
    // Slots of one quantisation group in both rings (token tiles up to 128): the lanes test the barriers of
    // the next kLook groups at once and the warp publishes every group up to the first one that is not ready,
    // so that what this warp costs per group (a test, a ballot, a release) is paid once per batch: a warp
    // that tests one barrier after the other needs about as long per group as the issuer does, and the two
    // then take turns instead of overlapping.
    constexpr bool kBatchedWatch = DEQUANT && kAGroup == 2 && kBGroup == 2;
    constexpr int kLook = kASlots < kBSlots ? kASlots : kBSlots;
    int gig = 0;                          // quantisation groups of this CTA's earlier units
    for (int u = blockIdx.x; kBatchedWatch && u < p.total_units && ok; u += gridDim.x, ++useq) {
      const Unit w = decode_unit(p, u, TOK);
      const int ngroups = (w.nkb + 1) >> 1;
      // the epilogue warps must have drained the previous unit's accumulator
      bool good = mbar_wait(bar_acc_empty, ((uint32_t)useq & 1u) ^ 1u, abort_flag, wait_limit);
      int done = 0;                       // groups of this unit published so far
      long long t0 = 0;
      bool timing = false;
      while (good && done < ngroups) {
        const int cand = done + lane;     // this lane's group of the unit
        bool rdy = false;
        if (lane < kLook && cand < ngroups) {
          // group gs uses slot gs % slots in round gs / slots of either ring; the groups of earlier rounds of a
          // slot lie before the head (kLook <= slots), so their phases are complete
          const int gs = gig + cand;
          rdy = mbar_test_wait(bar_a_deq(gs % kASlots), (uint32_t)(gs / kASlots) & 1u) &&
                mbar_test_wait(bar_b_full(gs % kBSlots), (uint32_t)(gs / kBSlots) & 1u);
        }
        const uint32_t mask = __ballot_sync(0xffffffffu, rdy);
        const int n = __ffs((int)~mask) - 1;            // consecutive ready groups from the head
        if (n > 0) {
          done += n;
          itg += 2 * n - ((done == ngroups && (w.nkb & 1)) ? 1 : 0);   // the last group of an odd K has one k-block
          if (lane == 0) st_release_shared(ready_addr, itg);
          timing = false;
        } else if (!timing) {
          t0 = clock64();
          timing = true;
        } else if (*abort_flag || clock64() - t0 > wait_limit) {
          good = false;
        }
      }
      if (!good) {
        if (lane == 0) st_release_shared(ready_addr, -1);
        ok = false;
        break;
      }
      gig += ngroups;
    }
    for (int u = blockIdx.x; !kBatchedWatch && u < p.total_units && ok; u += gridDim.x, ++useq) {
      const Unit w = decode_unit(p, u, TOK);
      for (int it = 0; it < w.nkb; ++it) {
        const int j = it % kAGroup;
        bool got = true;
        // the epilogue warps must have drained the previous unit's accumulator
        if (it == 0) got = mbar_wait(bar_acc_empty, ((uint32_t)useq & 1u) ^ 1u, abort_flag, wait_limit);
        if (DEQUANT && j == 0) got = got && mbar_wait(bar_a_deq(ra.s), ra.ph, abort_flag, wait_limit);
        if (it % kBGroup == 0) got = got && mbar_wait(bar_b_full(rb.s), rb.ph, abort_flag, wait_limit);
        __syncwarp();
        if (!got) {
          if (lane == 0) st_release_shared(ready_addr, -1);
          ok = false;
          break;
        }
        ++itg;
        if (lane == 0) st_release_shared(ready_addr, itg);
        if (j == kAGroup - 1 || it == w.nkb - 1) ra.next(kASlots);
        if (it % kBGroup == kBGroup - 1 || it == w.nkb - 1) rb.next(kBSlots);
      }
    }
    if (!ok) *abort_flag = 1;
  } else if (warp < kFirstDeqWarp) {
    // ------------------------------------------------------------------ scale warps
    if (DEQUANT) {
      const int sw = warp - kFirstScaleWarp;
      // seed and eps of the launch: its own, or those of the recorded step it belongs to
      const uint64_t seed = p.sp ? (uint64_t)p.sp->seed : p.seed;
      const float sign_eps = p.sp ? p.sign_eps * p.sp->eps : p.sign_eps;
      int gig = 0;                        // quantisation groups visited by this CTA so far (all units)
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u, TOK);
        const LinearDesc& L = p.lin[w.lin];
        const int ngroups = (w.nkb + 1) >> 1;
        for (int gi = 0; gi < ngroups; ++gi, ++gig) {
          if ((gig % kNumScaleWarps) != sw) continue;
          const int slot = gig % kNibSlots;              // the nibble-ring slot of this group
          const uint32_t gph = (uint32_t)(gig / kNibSlots) & 1u;
          const int r0 = lane * 4;                       // four consecutive output features = one counter block
          const bool live = w.n0 + r0 < L.N;             // N is a multiple of 8: all four or none
          // rows of scales of this slot: int4: the group's row; table mode: one row per k-block (block of 64 k)
          const int row0 = LUT ? w.kb_begin + 2 * gi : (w.kb_begin >> 1) + gi;
          const int rows = LUT ? min(2, w.nkb - 2 * gi) : 1;
          // token tiles never straddle pair_rows (checked on the host)
          const float se = (p.pair_rows > 0 && w.tok0 >= p.pair_rows) ? -sign_eps : sign_eps;
          // z does not depend on the stored scales: it is ready before they land
          float z[kScaleRows][4];
          uint2 raw[kScaleRows];
#pragma unroll
          for (int j = 0; j < kScaleRows; ++j) {
            z[j][0] = z[j][1] = z[j][2] = z[j][3] = 0.0f;
            raw[j] = make_uint2(0u, 0u);
            if (live && j < rows) {
              if (sign_eps != 0.0f) {
                const uint64_t i0 = L.idx_base + (uint64_t)((row0 + j) * p.scale_row_mul) * (uint64_t)L.N + (uint64_t)(w.n0 + r0);
                normals_of_block(seed, i0 >> 2, z[j]);
              }
              if (!Plan::kRawViaCopy) raw[j] = *reinterpret_cast<const uint2*>(L.scales + (size_t)((row0 + j) * p.scale_row_mul) * L.N + w.n0 + r0);
            }
          }
          uint8_t* const slot_mem = smem + Plan::kOffA + slot * Plan::kNibBytes;
          // kRawViaCopy: the stored scales came with the nibbles' copy; their arrival also says that the slot was
          // free.  Otherwise: the slot is free once the de-quantisers have read its previous group.
          const bool got = Plan::kRawViaCopy ? mbar_wait_relaxed(bar_nib_raw(slot), gph, abort_flag, wait_limit)
                                             : mbar_wait_relaxed(bar_nib_free(slot), gph ^ 1u, abort_flag, wait_limit);
          if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
#pragma unroll
          for (int j = 0; j < kScaleRows; ++j) {
            float sv[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (live && j < rows) {
              if (Plan::kRawViaCopy)
                raw[j] = *reinterpret_cast<const uint2*>(slot_mem + Plan::kOffRawInSlot + j * kRawScaleBytes + r0 * 2);
              const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw[j].x);
              const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw[j].y);
              sv[0] = fmaf(se, z[j][0], __low2float(a)); sv[1] = fmaf(se, z[j][1], __high2float(a));
              sv[2] = fmaf(se, z[j][2], __low2float(b)); sv[3] = fmaf(se, z[j][3], __high2float(b));
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
            uint4* dst = reinterpret_cast<uint4*>(slot_mem + Plan::kOffCookedInSlot + j * kCookedScaleBytes + r0 * 8);
            dst[0] = make_uint4(cooked[0], cooked[1], cooked[2], cooked[3]);
            dst[1] = make_uint4(cooked[4], cooked[5], cooked[6], cooked[7]);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_nib_full(slot));
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp < kFirstEpiWarp) {
    // ------------------------------------------------------------------ de-quantisers
    if (DEQUANT) {
      const int dt = threadIdx.x - kFirstDeqWarp * 32;      // 0 .. 128 kDeqTeams - 1
      const int r = (warp & 3) * 32 + lane;                 // row of the tile = TMEM lane this warp may access
      const int team = dt >> 7;                             // the teams of four warps take the groups in turn
      const __nv_bfloat162 magic_bias = __halves2bfloat162(__float2bfloat16_rn(136.0f), __float2bfloat16_rn(136.0f));
      __nv_bfloat162 s_hi, s_lo;
      *reinterpret_cast<uint32_t*>(&s_hi) = 0u;
      *reinterpret_cast<uint32_t*>(&s_lo) = 0u;
      // table mode: this lane's copy of the codebook (entry e at + 128 e)
      const uint32_t lut_lane = base + Plan::kOffLut + (uint32_t)lane * 4u;
      // nibbles of one 16-byte unit (32 consecutive k of this thread's row) -> 16 x bf16x2 (u - 8) * s', or
      // table[u] * s' in table mode
      auto dequant16 = [&](const uint4& pk, uint32_t (&outw)[16]) {
        const uint32_t words[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
          for (int pp = 0; pp < 4; ++pp) {
            __nv_bfloat162 q2;
            if (LUT) {
              const uint32_t x = (words[i] >> (4 * pp)) & 0x000F000Fu;             // codes of k = 2 j (low half) and 2 j + 1
              uint32_t ta, tb;
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(ta) : "r"(lut_lane + ((x & 0xFu) << 7)));
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tb) : "r"(lut_lane + (x >> 9)));      // (x >> 16) * 128
              const uint32_t t2 = (ta & 0x0000FFFFu) | (tb & 0xFFFF0000u);
              q2 = *reinterpret_cast<const __nv_bfloat162*>(&t2);
            } else {
              uint32_t x = ((words[i] >> (4 * pp)) & 0x000F000Fu) | 0x43004300u;   // bf16x2 {128 + u_lo, 128 + u_hi}
              q2 = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&x), magic_bias);     // exact u - 8
            }
            __nv_bfloat162 w2 = __hfma2(q2, s_hi, __hmul2(q2, s_lo));
            outw[i * 4 + pp] = *reinterpret_cast<uint32_t*>(&w2);                  // k = 32 h + 2 j, 2 j + 1 in register j
          }
        }
      };
      // A stage in tensor memory: lane = row (this warp's quadrant), column = k / 2
      const uint32_t a_lane_base = tmem_d + ((uint32_t)((warp & 3) * 32) << 16) + kAccCols;
      int gig = 0;                          // quantisation groups visited by this CTA so far (all units)
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u, TOK);
        for (int it = 0; it < w.nkb; it += 2, ++gig) {
          if ((gig % kDeqTeams) != team) continue;            // another team's group
          const int nslot = gig % kNibSlots;                  // nibble-ring slot of this group
          const uint32_t nph = (uint32_t)(gig / kNibSlots) & 1u;
          const int slot = gig % kASlots;                     // tensor-memory slot = one quantisation group (two k-blocks)
          const uint32_t gph = (uint32_t)(gig / kASlots) & 1u;
          const bool two = it + 1 < w.nkb;                    // the last group of an odd K has one k-block
          // the nibble slot is full: nibbles landed, perturbed scales written
          if (!__all_sync(0xffffffffu, mbar_wait(bar_nib_full(nslot), nph, abort_flag, wait_limit))) { ok = false; break; }
          const uint8_t* const slot_mem = smem + Plan::kOffA + nslot * Plan::kNibBytes;
          // perturbed scale of this row: one per group (int4) or one per k-block (table mode)
          uint2 cs[kScaleRows];
#pragma unroll
          for (int j = 0; j < kScaleRows; ++j)
            cs[j] = *reinterpret_cast<const uint2*>(slot_mem + Plan::kOffCookedInSlot + j * kCookedScaleBytes + r * 8);
          // this row's 64 k of each k-block: two 16-byte units (32 k each)
          const uint8_t* src = slot_mem + r * 16;
          uint4 pk[4];
          pk[0] = *reinterpret_cast<const uint4*>(src);
          pk[1] = *reinterpret_cast<const uint4*>(src + kTileN * 16);
          pk[2] = pk[3] = make_uint4(0, 0, 0, 0);
          if (two) {
            pk[2] = *reinterpret_cast<const uint4*>(src + kPackedTileBytes);
            pk[3] = *reinterpret_cast<const uint4*>(src + kPackedTileBytes + kTileN * 16);
          }
          // the slot's bytes are in registers: hand it back to the producer at once
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_nib_free(nslot));
          // the tensor-memory stages of the slot are free once the MMAs of their previous group retired
          if (!__all_sync(0xffffffffu, mbar_wait(bar_a_empty(slot), gph ^ 1u, abort_flag, wait_limit))) { ok = false; break; }
          tcgen05_fence_after();                              // orders the MMAs' reads of this slot before the stores below
          uint32_t outw[16];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            if (q4 < 2 || two) {
              if ((q4 & 1) == 0) {
                const uint2 c = cs[LUT ? (q4 >> 1) : 0];
                *reinterpret_cast<uint32_t*>(&s_hi) = c.x;
                *reinterpret_cast<uint32_t*>(&s_lo) = c.y;
              }
              dequant16(pk[q4], outw);
              tmem_st16(a_lane_base + (uint32_t)((slot * 2 + (q4 >> 1)) * kATmemColsPerStage + (q4 & 1) * 16), outw);
            }
          }
          tmem_wait_st();
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_a_deq(slot));
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == kStoreWarp) {
    // ------------------------------------------------------------------ store warp (bf16 tiles)
    // Walks the units and passes like the epilogue warps.  Two hardware barriers connect them in the
    // producer / consumer way: the epilogue warps sign "staged" (bar.arrive) when a pass sits in its
    // staging buffer and this warp waits for it (bar.sync); this warp signs "free" when the staging
    // buffer of a pass may be written and the epilogue warps wait for that.  Neither side waits for the
    // other's work: "free" for the next pass is signed before the store of this pass is issued (its
    // buffer was last read by the store issued two passes ago), so issuing a store, some hundred cycles,
    // runs beside the draining of the next pass.
    if (OUT_MODE == kOutBf16) {
      int useq = 0, sbuf = 0;
      bool store_pending = false, first = true;
      for (int u = blockIdx.x; u < p.total_units; u += gridDim.x, ++useq) {
        const Unit w = decode_unit(p, u, TOK);
        const CUtensorMap* tmap_y = w.lin == 0 ? &tmap_y0 : (w.lin == 1 ? &tmap_y1 : &tmap_y2);
        named_bar_sync(kBarUnit, kEpiBarThreads);           // the unit's accumulator is complete (or the wait for it failed)
        if (useq >= *epi_stop) break;
        for (int pass = 0; pass < Plan::kPasses; ++pass, sbuf = (sbuf + 1 == Plan::kStagingBufs) ? 0 : sbuf + 1) {
          const int tok_pass = w.tok0 + pass * Plan::kPassTok;
          if (tok_pass >= p.M) break;
          if (first) {                                      // all staging buffers start free
            named_bar_arrive(kBarFree, kEpiBarThreads);
            first = false;
          }
          named_bar_sync(kBarStaged, kEpiBarThreads);       // the pass is staged
          const bool more = (pass + 1 < Plan::kPasses && tok_pass + Plan::kPassTok < p.M) || u + (int)gridDim.x < p.total_units;
          if (more) {
            // the next pass's buffer was last read by the store issued two passes ago
            if (lane == 0 && store_pending) bulk_wait_group_read<Plan::kStagingBufs - 2>();
            __syncwarp();
            named_bar_arrive(kBarFree, kEpiBarThreads);
          }
          if (lane == 0) {
            tma_store_2d(tmap_y, base + Plan::kOffStaging + sbuf * Plan::kStagingBufBytes, w.n0, tok_pass);
            bulk_commit_group();
            store_pending = true;
          }
          __syncwarp();
        }
      }
      if (lane == 0 && store_pending) bulk_wait_group0();
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // TMEM lane = output feature, column = token.  Only the first epilogue warp polls the mbarrier;
    // the others are parked on a hardware barrier, which every epilogue warp reaches every time.
    // bf16 tiles: the store warp takes part in these barriers too.
    const int ew = warp - kFirstEpiWarp;
    const int quad = warp & 3;                          // TMEM lane quadrant this warp may read
    const int colpart = ew >> 2;                        // 0 or 1: which 16-column chunks this warp takes
    const int f = quad * 32 + lane;                     // feature within the tile
    const bool elected = (ew == 0 && lane == 0);
    constexpr int kChunksPerPass = Plan::kPassTok / 16;
    int useq = 0;
    int sbuf = 0;                                       // staging buffer of the next pass
    for (int u = blockIdx.x; u < p.total_units; u += gridDim.x, ++useq) {
      const Unit w = decode_unit(p, u, TOK);
      const LinearDesc& L = p.lin[w.lin];
      const int n = w.n0 + f;
      const float bias = (L.bias != nullptr && n < L.N && w.z == 0) ? L.bias[n] : 0.0f;
      if (ew == 0 && !mbar_wait(bar_acc_full, (uint32_t)useq & 1u, abort_flag, wait_limit)) {
        *epi_stop = useq;
        __threadfence_block();
      }
      named_bar_sync(kBarUnit, kEpiBarThreads);
      if (useq >= *epi_stop) { ok = false; break; }
      tcgen05_fence_after();
      if (OUT_MODE == kOutBf16) {
        // at most one 16-column chunk per warp and pass (kPassTok <= 32, two warps per lane quadrant)
        static_assert(kChunksPerPass <= 2, "one chunk per warp and pass");
        const bool mine = colpart < kChunksPerPass;
        // TMEM -> registers: this thread's feature for the 16 tokens of its chunk, as eight bf16 pairs
        auto load_pass = [&](int pass, uint32_t (&h)[8]) {
          if (mine) {
            uint32_t v[16];
            tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(pass * Plan::kPassTok + colpart * 16), v);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              h[j] = pack_bf16x2(__uint_as_float(v[2 * j]) + bias, __uint_as_float(v[2 * j + 1]) + bias);
          }
        };
        // registers -> staging buffer -> (store warp) TMA store
        auto stage_pass = [&](const uint32_t (&h)[8]) {
          unsigned short* const buf = reinterpret_cast<unsigned short*>(smem + Plan::kOffStaging +
                                                                        sbuf * Plan::kStagingBufBytes);
          named_bar_sync(kBarFree, kEpiBarThreads);         // the staging buffer of this pass may be written
          if (mine) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              buf[(colpart * 16 + 2 * j) * kTileN + f] = (unsigned short)(h[j] & 0xFFFFu);
              buf[(colpart * 16 + 2 * j + 1) * kTileN + f] = (unsigned short)(h[j] >> 16);
            }
          }
          fence_proxy_async_smem();                         // staged rows visible to the TMA store
          named_bar_arrive(kBarStaged, kEpiBarThreads);     // the store warp issues the pass's store
          sbuf = (sbuf + 1 == Plan::kStagingBufs) ? 0 : sbuf + 1;
        };
        // A full tile of at least four passes: the last half of the passes is first only read into
        // registers, so that the accumulator is handed back to the MMA warp before those passes are
        // staged and stored (the accumulator is single, its drain time is taken from the tensor pipe).
        constexpr int kHold = Plan::kPasses >= 4 ? Plan::kPasses / 2 : 0;
        if (kHold > 0 && w.tok0 + TOK <= p.M) {
          for (int pass = 0; pass < Plan::kPasses - kHold; ++pass) {
            uint32_t h[8];
            load_pass(pass, h);
            stage_pass(h);
          }
          uint32_t held[kHold > 0 ? kHold : 1][8];
#pragma unroll
          for (int k = 0; k < kHold; ++k) load_pass(Plan::kPasses - kHold + k, held[k]);
          tcgen05_fence_before();
          named_bar_sync(kBarDrained, kNumEpiWarps * 32);   // every epilogue warp has read its part of the accumulator
          if (elected) mbar_arrive(bar_acc_empty);          // the MMA warp may start the next unit
#pragma unroll
          for (int k = 0; k < kHold; ++k) stage_pass(held[k]);
          continue;
        }
        for (int pass = 0; pass < Plan::kPasses; ++pass) {
          const int tok_pass = w.tok0 + pass * Plan::kPassTok;
          if (tok_pass >= p.M) break;                       // uniform over the epilogue warps
          uint32_t h[8];
          load_pass(pass, h);
          if (pass == Plan::kPasses - 1 || tok_pass + Plan::kPassTok >= p.M) tcgen05_fence_before();
          stage_pass(h);
        }
        named_bar_sync(kBarDrained, kNumEpiWarps * 32);     // every epilogue warp has read its part of the accumulator
      } else {
        constexpr int kChunks = TOK / 16;
        for (int c = colpart; c < kChunks; c += 2) {
          if (w.tok0 + c * 16 >= p.M) break;                // warp-uniform
          uint32_t v[16];
          tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(c * 16), v);
          if (n < L.N) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int t = w.tok0 + c * 16 + j;
              if (t < p.M)
                reinterpret_cast<float*>(L.out)[((size_t)w.z * p.M + t) * L.ldo + n] = __uint_as_float(v[j]) + bias;
            }
          }
        }
        tcgen05_fence_before();
        named_bar_sync(kBarDrained, kNumEpiWarps * 32);
      }
      // accumulator drained: the MMA warp may start the next unit
      if (elected) mbar_arrive(bar_acc_empty);
    }
    if (!ok) *abort_flag = 1;
  }

  if (!ok && p.status != nullptr) atomicOr(p.status, kStatusTimeout);
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc(tmem_d, kTmemCols);
  }
}

// Sum of split-K partials in a fixed order, + bias, to bf16.
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int splits, int M, int N,
                                     const float* __restrict__ bias, __nv_bfloat16* __restrict__ out, int ldo) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)M * N) return;
  const int t = (int)(idx / N), n = (int)(idx % N);
  float acc = 0.0f;
  for (int z = 0; z < splits; ++z) acc += part[((size_t)z * M + t) * N + n];
  if (bias) acc += bias[n];
  out[(size_t)t * ldo + n] = __float2bfloat16_rn(acc);
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

// 2-D bf16 tensor map of a row-major [rows][ld] matrix of which `cols` columns are addressed;
// box = box_cols x box_rows.  Operand tiles use the 128-byte swizzle (box_cols = 64); output
// tiles are plain rows of 128 features.
int make_tmap_bf16(CUtensorMap* map, const void* ptr, int rows, int cols, int ld, int box_cols, int box_rows,
                   bool swizzle128) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return QZO_ERR_CUDA;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QZO_OK : QZO_ERR_CUDA;
}

int pick_tok_tile(int M) {
  if (M <= 16) return 16;
  if (M <= 32) return 32;
  if (M <= 64) return 64;
  if (M <= 128) return 128;
  return 256;
}

// SMs of the current device (cached per device id).
int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int n = cached[dev].load();
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n);
  }
  return n;
}

template <int TOK, int WMODE, int OUT_MODE>
int launch_one(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap* ty, const GemmParams& p,
               cudaStream_t st) {
  using Plan = SmemPlan<TOK, WMODE, OUT_MODE>;
  auto kern = w4a16_gemm_kernel<TOK, WMODE, OUT_MODE>;
  static std::atomic<unsigned long long> configured{0};      // per instantiation, one bit per device
  if (first_use_on_device(configured))
    QZO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan::kDynamicBytes));
  const int grid = p.total_units < sm_count() ? p.total_units : sm_count();
  QZO_LAUNCH(kern, dim3(grid), dim3(Roles<TOK, WMODE>::kThreads), Plan::kDynamicBytes, st, tx, tw, ty[0], ty[1], ty[2], p);
  return QZO_OK;
}

template <int WMODE, int OUT_MODE>
int launch_tok(int tok, const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap* ty, const GemmParams& p,
               cudaStream_t st) {
  switch (tok) {
    case 16: return launch_one<16, WMODE, OUT_MODE>(tx, tw, ty, p, st);
    case 32: return launch_one<32, WMODE, OUT_MODE>(tx, tw, ty, p, st);
    case 64: return launch_one<64, WMODE, OUT_MODE>(tx, tw, ty, p, st);
    case 128: return launch_one<128, WMODE, OUT_MODE>(tx, tw, ty, p, st);
    default: return launch_one<256, WMODE, OUT_MODE>(tx, tw, ty, p, st);
  }
}

}  // namespace

// Test hook of the bounded waits (see qzo_debug_gemm_wait_expiry): a shorter wait limit and a group whose copies
// are withheld, for the launches of the calling thread while the hook is set.
static thread_local long long g_debug_wait_limit = 0;
static thread_local int g_debug_skip_group = -1;
void set_gemm_wait_debug(long long limit_cycles, int skip_group) {
  g_debug_wait_limit = limit_cycles > kWaitLimitCycles ? kWaitLimitCycles : limit_cycles;
  g_debug_skip_group = skip_group;
}

// Split-K plan: number of K slices for a problem (1 = none).  Slices hold an even number of
// k-blocks so that they start on a quantisation-group boundary.  The choice minimises a simple
// cost model measured on B200: a unit costs a pipeline fill plus ~600 cycles per k-block whatever
// the token tile, the units run in rounds of one per SM, and a split adds the fp32 partial sums'
// round trip and a second launch.  Depends on the shape only, so results are reproducible.
static int gemm_splits_tok(int M, int K, int N, int tok) {
  if (tok > 128) return 1;                       // 256-token tiles: plenty of units, tensor-bound
  const int tiles = ceil_div(N, kTileN) * ceil_div(M, tok);
  const int groups = ceil_div(K, kGroup);
  const int sms = sm_count();                    // of the current device (148 on B200)
  const double cycles_per_kb = 600.0, fill_cycles = 3500.0, clock_ghz = 1.8;
  int best = 1;
  double best_us = 1e30;
  for (int sp = 1; sp <= 16 && sp <= groups; ++sp) {
    const int groups_per = ceil_div(groups, sp);
    if (sp > 1 && groups_per < 4) break;         // at least four groups per slice
    const int slices = ceil_div(groups, groups_per);
    if (slices != sp) continue;                  // same partition as a smaller sp
    const int rounds = ceil_div(tiles * slices, sms);
    double us = rounds * (groups_per * 2 * cycles_per_kb + fill_cycles) / (clock_ghz * 1e3);
    if (sp > 1) us += 3.0 + (double)(sp + 1) * M * N * 4.0 / 3.0e6;   // second launch + partial sums at ~3 TB/s
    if (us < best_us) { best_us = us; best = sp; }
  }
  return best;
}

int gemm_splits(int M, int K, int N) { return gemm_splits_tok(M, K, N, pick_tok_tile(M)); }

// Token tile of a launch over M rows.  A launch that switches the perturbation sign at row `pair_rows`
// (M = 2 pair_rows) takes the tile of pair_rows rows and needs pair_rows to be a multiple of it, so that
// the boundary falls between two token tiles and the launch has exactly the units of the two single-sign
// launches it replaces: pair_rows in {16, 32, 64, 128} or a multiple of 256; 0 otherwise.
static int launch_tok_tile(int M, int pair_rows) {
  if (pair_rows <= 0) return pick_tok_tile(M);
  const int t = pick_tok_tile(pair_rows);
  return pair_rows % t == 0 ? t : 0;
}

bool paired_rows_ok(int M, int pair_rows) {
  return pair_rows > 0 && pair_rows < M && launch_tok_tile(M, pair_rows) > 0;
}

size_t gemm_workspace_bytes(int M, int K, int N, int pair_rows) {
  const int tok = launch_tok_tile(M, pair_rows);
  const int splits = tok > 0 ? gemm_splits_tok(pair_rows > 0 ? pair_rows : M, K, N, tok) : 1;
  if (splits <= 1) return 0;
  return (size_t)splits * M * N * sizeof(float);
}

// Y_j = X W'_j (+ bias_j) for up to three linears that share X, with W'_j de-quantised
// from int4 and perturbed scales.
// pair_rows > 0: rows [0, pair_rows) are perturbed with sign * eps, rows [pair_rows, M) with -sign * eps;
// see paired_rows_ok for the row counts that allow it.
// lut16 (host, 16 floats) non-null: table mode: the nibbles index that table and the scales are [ceil(K/64)][N], one
// row per block of 64 k; null: int4 with one row of scales per group of 128 k.
// d_sp (device) non-null: seed and eps are read from it when the kernel runs, the arguments of those names are ignored.
// channel_scales: the scales are one row [N] for all k (channel-wise), index idx_base + n.
int launch_perturbed_gemm_group(const __nv_bfloat16* d_x, int M, int K, const GemmLinear* lins, int n_lin,
                                uint64_t seed, int sign, float eps, int pair_rows, void* d_ws, size_t ws_bytes,
                                int* d_status, cudaStream_t st, const float* lut16, const StepParams* d_sp, bool channel_scales) {
  if (M <= 0 || K <= 0 || (K % 8) != 0 || n_lin < 1 || n_lin > kMaxGroupedLinears) return QZO_ERR_BAD_ARG;
  if (pair_rows != 0 && !paired_rows_ok(M, pair_rows)) return QZO_ERR_BAD_ARG;
  for (int j = 0; j < n_lin; ++j)
    if (lins[j].N <= 0 || (lins[j].N % 8) != 0 || (lins[j].idx_base % 4) != 0 || (lins[j].ldo % 8) != 0)
      return QZO_ERR_BAD_ARG;
  const int tok = launch_tok_tile(M, pair_rows);
  // A paired launch slices K like each of the two single-sign launches it replaces, so that both ways of
  // running a step add up the same partial sums in the same order.
  const int m_plan = pair_rows > 0 ? pair_rows : M;
  // split-K only pays for small token counts; grouped launches of such problems go one by one
  if (n_lin > 1) {
    bool any_split = false;
    for (int j = 0; j < n_lin; ++j) any_split = any_split || gemm_splits_tok(m_plan, K, lins[j].N, tok) > 1;
    if (any_split) {
      for (int j = 0; j < n_lin; ++j)
        QZO_TRY(launch_perturbed_gemm_group(d_x, M, K, lins + j, 1, seed, sign, eps, pair_rows, d_ws, ws_bytes, d_status,
                                            st, lut16, d_sp, channel_scales));
      return QZO_OK;
    }
  }
  CUtensorMap tx, ty[kMaxGroupedLinears];
  QZO_TRY(make_tmap_bf16(&tx, d_x, M, K, K, kBlockK, tok, true));
  GemmParams p{};
  p.n_lin = n_lin;
  p.M = M; p.K = K;
  p.num_kb = ceil_div(K, kBlockK);
  p.m_tiles = ceil_div(M, tok);
  p.seed = seed;
  p.sign_eps = d_sp ? (float)sign : (float)sign * eps;
  p.sp = d_sp;
  p.pair_rows = pair_rows;
  p.status = d_status;
  p.wait_limit = g_debug_wait_limit > 0 ? g_debug_wait_limit : kWaitLimitCycles;
  p.skip_group = g_debug_skip_group;
  p.scale_row_mul = channel_scales ? 0 : 1;
  if (lut16) memcpy(p.lut, lut16, sizeof(p.lut));
  const int splits = (n_lin == 1) ? gemm_splits_tok(m_plan, K, lins[0].N, tok) : 1;
  for (int j = 0; j < n_lin; ++j) {
    LinearDesc& L = p.lin[j];
    L.wq = reinterpret_cast<const uint8_t*>(lins[j].wq);
    L.scales = lins[j].scales;
    L.idx_base = lins[j].idx_base;
    L.N = lins[j].N;
    L.n_tiles = ceil_div(lins[j].N, kTileN);
    p.tiles_n_total += L.n_tiles;
    if (splits <= 1) {
      L.bias = lins[j].bias; L.out = lins[j].out; L.ldo = lins[j].ldo;
    }
  }
  if (splits <= 1) {
    for (int j = 0; j < kMaxGroupedLinears; ++j) {
      const GemmLinear& g = lins[j < n_lin ? j : 0];
      QZO_TRY(make_tmap_bf16(&ty[j], g.out, M, g.N, g.ldo, kTileN, tok < 32 ? tok : 32, false));
    }
    p.splits = 1;
    p.kb_per_split = ceil_div(p.num_kb, 2) * 2;
    p.total_units = p.tiles_n_total * p.m_tiles;
    return lut16 ? launch_tok<kWTable16, kOutBf16>(tok, tx, tx, ty, p, st) : launch_tok<kWInt4, kOutBf16>(tok, tx, tx, ty, p, st);
  }
  const GemmLinear& g = lins[0];
  const int groups = ceil_div(K, kGroup);
  const size_t need = (size_t)splits * M * g.N * sizeof(float);
  if (d_ws == nullptr || ws_bytes < need) return QZO_ERR_WORKSPACE;
  const int groups_per = ceil_div(groups, splits);
  const int zdim = ceil_div(groups, groups_per);           // every slice is non-empty
  p.lin[0].bias = nullptr; p.lin[0].out = d_ws; p.lin[0].ldo = g.N;
  p.splits = zdim;
  p.kb_per_split = groups_per * 2;
  p.total_units = p.tiles_n_total * p.m_tiles * zdim;
  ty[0] = ty[1] = ty[2] = tx;                              // unused by the fp32 epilogue
  if (lut16) QZO_TRY((launch_tok<kWTable16, kOutF32>(tok, tx, tx, ty, p, st)));
  else QZO_TRY((launch_tok<kWInt4, kOutF32>(tok, tx, tx, ty, p, st)));
  const int64_t total = (int64_t)M * g.N;
  QZO_LAUNCH(splitk_reduce_kernel, dim3((unsigned)ceil_div64(total, 256)), dim3(256), 0, st,
             reinterpret_cast<const float*>(d_ws), zdim, M, g.N, g.bias, g.out, g.ldo);
  return QZO_OK;
}

// logits[t][v] = sum_k X[t][k] Wh[v][k]: bf16 weights [V][K] row-major, fp32 output [M][V].
int launch_bf16_gemm_f32out(const __nv_bfloat16* d_x, const __nv_bfloat16* d_w, float* d_out, int M, int K, int N,
                            int* d_status, cudaStream_t st) {
  if (M <= 0 || K <= 0 || N <= 0 || (K % 8) != 0) return QZO_ERR_BAD_ARG;
  const int tok = pick_tok_tile(M);
  CUtensorMap tx, tw, ty[kMaxGroupedLinears];
  QZO_TRY(make_tmap_bf16(&tx, d_x, M, K, K, kBlockK, tok, true));
  QZO_TRY(make_tmap_bf16(&tw, d_w, N, K, K, kBlockK, kTileN, true));
  ty[0] = ty[1] = ty[2] = tx;                              // unused by the fp32 epilogue
  GemmParams p{};
  p.n_lin = 1;
  p.lin[0].N = N; p.lin[0].ldo = N; p.lin[0].out = d_out; p.lin[0].n_tiles = ceil_div(N, kTileN);
  p.tiles_n_total = p.lin[0].n_tiles;
  p.M = M; p.K = K;
  p.num_kb = ceil_div(K, kBlockK);
  p.kb_per_split = ceil_div(p.num_kb, 2) * 2;
  p.splits = 1;
  p.m_tiles = ceil_div(M, tok);
  p.total_units = p.tiles_n_total * p.m_tiles;
  p.status = d_status;
  p.wait_limit = kWaitLimitCycles;
  p.skip_group = -1;
  return launch_tok<kWBf16, kOutF32>(tok, tx, tw, ty, p, st);
}

}  // namespace qzo

// ------------------------------------------------------------------------------------------
// Entry point that allocates nothing: the split-K partial sums live in a fixed array inside
// the library image instead of a caller-provided workspace.
// ------------------------------------------------------------------------------------------
namespace {

// Scratch of the allocation-free entry point.  One copy per device that loads the library,
// held until the process exits.  In host code this name is only a handle for the symbol, not a
// device address: the address is resolved per device below and passed to the kernels.
static __device__ __align__(256) unsigned char g_noalloc_scratch[QZO_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (resolved once per device).
int noalloc_scratch_address(void** out) {
  int dev = 0;
  QZO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return QZO_ERR_UNSUPPORTED_DEVICE;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (g_noalloc_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    QZO_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    if (ptr == nullptr) return QZO_ERR_CUDA;
    g_noalloc_ptr[dev] = ptr;
  }
  *out = g_noalloc_ptr[dev];
  return QZO_OK;
}

}  // namespace

extern "C" int qzo_perturbed_gemm_noalloc(const void* d_x_bf16, const void* d_wq, const void* d_scales_bf16,
                                          const float* d_bias, void* d_y_bf16, int M, int K, int N, uint64_t seed,
                                          uint64_t scale_index_base, int sign, float eps, int* d_status,
                                          void* stream) {
  if (!d_x_bf16 || !d_wq || !d_scales_bf16 || !d_y_bf16) return QZO_ERR_BAD_ARG;
  if (M <= 0 || K <= 0 || N <= 0 || (N % 8) || (K % 8)) return QZO_ERR_BAD_ARG;
  if (sign < -1 || sign > 1 || !(eps > 0.0f)) return QZO_ERR_BAD_ARG;
  if (((uintptr_t)d_x_bf16 & 15) || ((uintptr_t)d_wq & 15) || ((uintptr_t)d_scales_bf16 & 15) ||
      ((uintptr_t)d_y_bf16 & 15))
    return QZO_ERR_BAD_ARG;
  // a problem whose partial sums do not fit the fixed array is refused, never truncated
  if (qzo::gemm_workspace_bytes(M, K, N) > (size_t)QZO_NOALLOC_SCRATCH_BYTES) return QZO_ERR_WORKSPACE;
  QZO_TRY(qzo::check_device());
  void* scratch = nullptr;
  QZO_TRY(noalloc_scratch_address(&scratch));
  const qzo::GemmLinear g{d_wq, (const __nv_bfloat16*)d_scales_bf16, d_bias, (__nv_bfloat16*)d_y_bf16, N, N,
                          scale_index_base};
  return qzo::launch_perturbed_gemm_group((const __nv_bfloat16*)d_x_bf16, M, K, &g, 1, seed, sign, eps, 0, scratch,
                                          (size_t)QZO_NOALLOC_SCRATCH_BYTES, d_status, (cudaStream_t)stream);
}

