// Integer GEMM on quantization codes with the de-quantizing epilogue, for sm_100a.
//
//   acc[m][n] = sum_k xq[m][k] * wq[n][k]      tcgen05.mma kind::i8, int32 accumulators in TMEM
//   z = fma(float(acc) * s_x, s_w[n], bias[n]);  y = residual + residual_scale * act(z)
//
// One persistent CTA per SM walks output tiles of 128 x BN.  Warp roles:
//   warp 0        TMA producer: A (activation codes) and B (weight codes) k-blocks of 128 bytes
//                 into a ring of shared-memory stages, 128-byte swizzled, K-major
//   warp 1        MMA issuer: one thread issues four K=32 MMAs per k-block into one of two TMEM
//                 accumulator buffers and commits the stage back to the producer
//   warps 2..     epilogue (4, 8 or 16 warps): TMEM -> registers -> de-quantize / bias / activation / residual ->
//                 swizzled shared staging -> TMA store; overlaps the next tile's MMAs.  The
//                 residual tile is fetched by TMA into the same staging buffer beforehand.
// CTA pairs (K > 512, M > 128): two CTAs of a cluster share one 256-row tile.  Each loads its own
// 128 rows of A and half of the tile's weight rows; the pair's leader issues
// tcgen05.mma.cta_group::2 (M = 256), which reads both CTAs' shared memory and writes each CTA's
// rows into that CTA's TMEM.  Per CTA this halves the weight bytes per MMA clock (operand loads and
// shared-memory reads), which is what bounds the deep-K shapes.  No load is multicast.
// Every wait on an mbarrier is bounded by a wall-clock limit; on expiry the CTA records
// AQT_ERR_TIMEOUT in the device status word, leaves its loops, frees its TMEM and returns.
#pragma once

#include <cuda.h>
#include <string.h>

#include "aqt_common.cuh"
#include "pack.cuh"
#include "row_quant_epilogue.cuh"

namespace aqt {

constexpr int kBM = 128;         // tile rows = TMEM lanes
constexpr int kBK = 128;         // bytes (= int8 elements) of K per pipeline stage: one swizzle row
constexpr int kMmaK = 32;        // K of one tcgen05.mma kind::i8
constexpr int kStoreBoxRows = 32;
constexpr int kStoreBoxCols = 32;                                  // fp32: 128 bytes = one swizzle row
constexpr int kStageBufBytes = kStoreBoxRows * kStoreBoxCols * 4;  // 4 KB
constexpr uint64_t kWaitLimitNs = 2000000000ull;                   // 2 s

// BN: tile width.  STAGES: depth of the operand ring.  EW: epilogue warps, 4, 8 or 16 (one, two or
// four per TMEM lane quadrant, each taking an equal share of the tile's columns).  Shallow-K
// shapes are bound by the epilogue (special-function and issue throughput, long dependent chains)
// and take 8 or 16 warps; deep-K shapes are bound by operand loads and give the shared memory of
// the extra staging buffers to the ring.
// WS ("weight stationary", K <= 512): a CTA keeps one n-tile of the weights resident in shared
// memory for its whole life and streams only activation k-blocks through the ring, which halves
// the L2 -> shared-memory traffic and lets the ring hold more than one tile of A.
constexpr int kWsMaxKBlocks = 4;  // K <= 512
template <int BN, int STAGES, int EW, bool WS, bool CTA2 = false>
struct GemmCfg {
  static_assert(!(WS && CTA2), "the weight-stationary kernel runs one CTA per tile");
  static constexpr int kThreads = 32 * (2 + EW);
  static constexpr int kABytes = kBM * kBK;
  static constexpr int kBBytes = (CTA2 ? BN / 2 : BN) * kBK;  // a CTA of a pair holds half of the tile's weight rows
  static constexpr int kStageBytes = WS ? kABytes : kABytes + kBBytes;
  static constexpr int kResidentBytes = WS ? kWsMaxKBlocks * kBBytes : 0;
  static constexpr int kStages = STAGES;
  // Two accumulator buffers, so that the epilogue of a tile overlaps the next tile's MMAs; a tile
  // 512 columns wide (CTA pairs only) fills tensor memory by itself and has one.
  static_assert(BN <= 256 || (BN == 512 && CTA2), "512-column tiles are a form of the CTA-pair kernel");
  static constexpr int kAccBufs = BN == 512 ? 1 : 2;
  static constexpr int kMmaN = BN > 256 ? 256 : BN;  // columns one tcgen05.mma covers
  static constexpr int kTmemCols = kAccBufs * BN;    // a power of two >= 32
  // Output staging buffers per warp: two let a warp fill one while the bulk store of the other is
  // still being read; with sixteen warps each warp stores once per tile and one is enough.
  // "Lean" epilogue: where the ring, two staging buffers per warp and the scale slabs together
  // would not fit (a fourth ring stage bought with eight epilogue warps), a warp keeps one staging
  // buffer and reads scales and biases through L1.  A load takes about 2200 clocks from issue to
  // arrival, so the ring depth sets the k-block rate: three stages give 705 clocks per k-block
  // against 554 of MMA time, four give the MMA rate.
  static constexpr bool kLean = !WS && EW == 8 &&
                                STAGES * kStageBytes + EW * 2 * kStageBufBytes + EW * 2 * (BN / (EW / 4)) * 4 + 1024 + 512 > 232448;
  static constexpr int kStageBufs = (EW == 16 || kLean) ? 1 : 2;
  static constexpr int kEpiBytes = EW * kStageBufs * kStageBufBytes;
  // Scales and biases of the tile's columns in shared memory: one slab per CTA when the n-tile is
  // fixed (WS), one per warp (its own columns) with EW >= 8 otherwise; with EW == 4 they are read
  // through L1 instead (the epilogue is a small part of a deep-K tile).
  static constexpr bool kScaleSlab = WS || (EW >= 8 && !kLean);
  static constexpr int kSlabFloats = WS ? BN : BN / (EW / 4);  // per array (s_w, bias)
  static constexpr int kScaleBytes = !kScaleSlab ? 0 : (WS ? 2 * BN * 4 : EW * 2 * kSlabFloats * 4);
  static constexpr int kSmemBytes = STAGES * kStageBytes + kResidentBytes + kEpiBytes + kScaleBytes + 1024;  // + alignment slack
  static_assert(kSmemBytes + 512 <= 232448, "ring + resident weights + staging must fit the 227 KB a CTA can opt into");
  static_assert(!WS || kWsMaxKBlocks * BN * 64 <= kEpiBytes, "packed weights are staged in the epilogue buffers");
};

struct GemmParams {
  const float* s_x;
  const float* s_w;
  const float* bias;
  const float* residual;
  int32_t* acc_debug;
  int64_t ldr;
  float residual_scale;
  int s_x_kind;
  int act;
  int M, N, K;  // K: bytes of contraction per operand row (= elements for 8-bit codes, 4 x elements for the float kind)
  int kind = 0;       // 0: signed 8-bit codes, int32 accumulators; 1: binary32 operands used as tf32, binary32 accumulators
  int64_t a_pitch = 0;  // bytes between rows of A; 0 = dense (K)
  // Batched form (streaming kernel, one CTA per tile): every batch_tiles_m consecutive m-tiles form
  // one batch with its own block of batch_b_rows rows of B, stacked below one another (b_rows rows
  // in all; 0 = N).  Used to split a very deep contraction over CTAs: batch s holds the s-th
  // chunk of the contraction of both operands, and the batches' outputs are added afterwards.
  int batch_tiles_m = 0;
  int batch_b_rows = 0;
  int64_t b_rows = 0;
  int n_out;    // N, or N / 2 for the GLU forms
  int tiles_m, tiles_n, k_blocks;
  int small_acc;  // every |accumulator| < 2^22: the int -> float conversion can use the exponent trick
  // Row-quantizing epilogue (template argument RQ of the CTA-pair kernel): the output rows leave the
  // kernel as codes and scales as well (or only), see the kernel.
  uint8_t* q_out = nullptr;         // int8 codes [M, N], dense
  float* s_out = nullptr;           // [M] row scales
  uint64_t* exchange = nullptr;     // [rows padded to the tile height][exchange_parts] words: (tag << 32) | bits of a part's row maximum
  uint32_t* generation = nullptr;   // [groups] counters that make the tag differ on every execution
  uint32_t tag = 0;                 // tag of this call
  int exchange_parts = 0;           // column parts a row's maximum is assembled from: tiles_n x warps per lane quadrant
  int qmax_out = 127;
  int rounding = AQT_ROUND_NEAREST_EVEN;
  int has_y = 1;                    // 0: no fp32 output
  // The weights (codes, scales, bias) were complete before the kernel ahead of this one in the stream
  // was enqueued, so a kernel may read them before that kernel has finished (see grid_dependency_wait).
  int static_w = 0;
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One attempt.  The thread may stay suspended in the instruction for up to kTryWaitSuspendNs while
// the phase is incomplete (it resumes at once when the phase completes), so a waiting warp costs
// its scheduler a handful of instructions per 100 us instead of a spin loop's worth: the producer,
// the MMA issuer and the exchange warp share their schedulers with the epilogue warps.
constexpr uint32_t kTryWaitSuspendNs = 100000u;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity), "r"(kTryWaitSuspendNs)
      : "memory");
  return done != 0;
}

// Bounded wait.  Returns false if the CTA is aborting or the limit passed (and then sets both
// the CTA's abort flag and the device status word).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint64_t t_start,
                                          uint64_t limit_ns = kWaitLimitNs) {
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 0x3) == 0) {  // an attempt can last kTryWaitSuspendNs: look at the clock every few
      if (*abort_flag) return false;
      if (global_timer_ns() - t_start > limit_ns) {
        *abort_flag = 1;
        atomicExch(&g_device_status, AQT_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 2-D tiled load into this CTA's shared memory, completion counted in bytes on `bar`.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* m, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
// The same for a CTA of a pair: completion is counted on the barrier at the same shared-memory
// offset in the pair's leader (rank bit of the address cleared).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(c0), "r"(c1), "r"(bar & 0xFEFFFFFFu)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the mbarrier at this shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(bar), "r"(rank));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Pair form: arrive on the barrier at this offset in both CTAs once the pair's MMAs have completed.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"((uint16_t)3)
               : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T, 256 x N x 32: each CTA supplies 128 rows of A and N/2 rows of B.
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on an mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x N x 32, signed 8-bit operands, int32 accumulate.
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The float forms: A and B hold binary32 values of which the tensor core uses sign, exponent and
// the upper ten fraction bits (tf32); products are summed into binary32 accumulators.  One
// instruction covers K = 8 elements = 32 bytes, so operand tiles, swizzle and the descriptor
// advance are byte-for-byte those of the 8-bit kind.
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_mma_tf32_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (base + i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand tile whose rows are 128 bytes, stored with the
// 128-byte swizzle (what the TMA load writes); 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                    // leading-dimension offset: not used by swizzled K-major
  d |= (uint64_t)(1024 >> 4) << 32;          // stride between 8-row groups
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}
// Instruction descriptor: D int32, A and B signed 8-bit, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t idesc_i8(int bn, int m = kBM) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
// The same for the float kind: D binary32, A and B tf32, both K-major.
__host__ __device__ constexpr uint32_t idesc_tf32(int bn, int m = kBM) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// Epilogue math

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// sigmoid(z) = 1 / (1 + e^-z) with e^-z = 2^(-z log2 e): one multiply, the special-function
// unit's 2^t, one add, its reciprocal.  Five instructions with the caller's final multiply, two of
// them on the special-function unit, which is the unit that bounds the Swish epilogue.
// Error: |t| 7e-8 from the rounded product, 2^-22 from 2^t, 2^-23 from the reciprocal; relative to
// the pre-activation |z| the activation a = z sigmoid(z) is within 3e-7 everywhere (the relative
// error of a itself passes 1e-6 only below z = -9, where |a| < 1e-3 |z|).  Large |t| saturates
// cleanly: 2^t = +inf gives sigmoid 0, 2^t = 0 gives sigmoid 1.
__device__ __forceinline__ float sigmoid_f(float z) {
  const float e = ex2_approx(z * -1.4426950408889634f);
  return rcp_approx(1.0f + e);
}

// What a TMEM accumulator word holds and how it becomes a float (template argument ACCK):
//   kAccInt32      int32, converted round-to-nearest-even (exact below 2^24)
//   kAccInt32Small int32 with |acc| < 2^22 guaranteed by the caller: adding the integer to the bit
//                  pattern of 1.5 * 2^23 and subtracting that constant is exact and stays off the
//                  conversion unit
//   kAccFloat      binary32 already (the float matmul of the weight-only layer)
constexpr int kAccInt32 = 0, kAccInt32Small = 1, kAccFloat = 2;
template <int ACCK>
__device__ __forceinline__ float acc_to_float(uint32_t acc) {
  if (ACCK == kAccFloat) return __uint_as_float(acc);
  if (ACCK == kAccInt32Small) return __int_as_float(0x4B400000 + (int)acc) - 12582912.0f;
  return __int2float_rn((int)acc);
}

// Two accumulators -> two floats (see acc_to_float); the subtraction is one packed add.
template <int ACCK>
__device__ __forceinline__ float2 acc_to_float2(uint32_t a0, uint32_t a1) {
  if (ACCK == kAccFloat) return make_float2(__uint_as_float(a0), __uint_as_float(a1));
  if (ACCK == kAccInt32Small)
    return __fadd2_rn(make_float2(__int_as_float(0x4B400000 + (int)a0), __int_as_float(0x4B400000 + (int)a1)),
                      make_float2(-12582912.0f, -12582912.0f));
  return make_float2(__int2float_rn((int)a0), __int2float_rn((int)a1));
}

// z[i] = fma(float(acc[i]) * sx, s_w[i], bias[i]) for 32 consecutive columns whose scales and
// biases sit at `sw_smem` / `b_smem` (shared-memory byte addresses, 16-byte aligned).  The
// arithmetic runs on the packed two-lane fp32 instructions of this architecture (each lane an
// ordinary round-to-nearest IEEE operation), which halves the issue slots it takes.
template <int ACCK>
__device__ __forceinline__ void dequant32(const uint32_t (&acc)[32], float sx, uint32_t sw_smem, uint32_t b_smem, float (&z)[32]) {
  const float2 sx2 = make_float2(sx, sx);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float w0, w1, w2, w3, b0, b1, b2, b3;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(w0), "=f"(w1), "=f"(w2), "=f"(w3) : "r"(sw_smem + 16 * j));
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(b0), "=f"(b1), "=f"(b2), "=f"(b3) : "r"(b_smem + 16 * j));
    const float2 z01 = __ffma2_rn(__fmul2_rn(acc_to_float2<ACCK>(acc[4 * j + 0], acc[4 * j + 1]), sx2), make_float2(w0, w1), make_float2(b0, b1));
    const float2 z23 = __ffma2_rn(__fmul2_rn(acc_to_float2<ACCK>(acc[4 * j + 2], acc[4 * j + 3]), sx2), make_float2(w2, w3), make_float2(b2, b3));
    z[4 * j + 0] = z01.x;
    z[4 * j + 1] = z01.y;
    z[4 * j + 2] = z23.x;
    z[4 * j + 3] = z23.y;
  }
}

// a[i] = a[i] * sigmoid(a[i]) (see sigmoid_f) for 32 values, two per instruction where the
// operation is an IEEE multiply or add.
__device__ __forceinline__ void swish32(float (&a)[32]) {
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float2 z = make_float2(a[2 * j], a[2 * j + 1]);
    const float2 t = __fmul2_rn(z, make_float2(-1.4426950408889634f, -1.4426950408889634f));
    const float2 d = __fadd2_rn(make_float2(1.0f, 1.0f), make_float2(ex2_approx(t.x), ex2_approx(t.y)));
    const float2 y = __fmul2_rn(z, make_float2(rcp_approx(d.x), rcp_approx(d.y)));
    a[2 * j] = y.x;
    a[2 * j + 1] = y.y;
  }
}

__device__ __forceinline__ float4 ld4_guard(const float* base, int n, int limit) {
  if (base == nullptr) return make_float4(0.f, 0.f, 0.f, 0.f);
  if (n + 3 < limit) return __ldg(reinterpret_cast<const float4*>(base + n));
  float4 r;
  r.x = n + 0 < limit ? __ldg(base + n + 0) : 0.f;
  r.y = n + 1 < limit ? __ldg(base + n + 1) : 0.f;
  r.z = n + 2 < limit ? __ldg(base + n + 2) : 0.f;
  r.w = n + 3 < limit ? __ldg(base + n + 3) : 0.f;
  return r;
}

// The same with scales and biases read from global memory (warp-uniform addresses, served by L1).
template <int ACCK>
__device__ __forceinline__ void dequant32_gmem(const uint32_t (&acc)[32], float sx, const float* s_w, const float* bias, int n0,
                                               int limit, float (&z)[32]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float4 w = ld4_guard(s_w, n0 + 4 * j, limit);
    const float4 b = ld4_guard(bias, n0 + 4 * j, limit);
    z[4 * j + 0] = __fmaf_rn(__fmul_rn(acc_to_float<ACCK>(acc[4 * j + 0]), sx), w.x, b.x);
    z[4 * j + 1] = __fmaf_rn(__fmul_rn(acc_to_float<ACCK>(acc[4 * j + 1]), sx), w.y, b.y);
    z[4 * j + 2] = __fmaf_rn(__fmul_rn(acc_to_float<ACCK>(acc[4 * j + 2]), sx), w.z, b.z);
    z[4 * j + 3] = __fmaf_rn(__fmul_rn(acc_to_float<ACCK>(acc[4 * j + 3]), sx), w.w, b.w);
  }
}

// ------------------------------------------------------------------------------------------------
// The kernel

// i-th tile of this CTA.  Standard order: tiles are numbered n-fastest and dealt round-robin.
// Weight-stationary order: the CTA owns n-tile (blockIdx % tiles_n) and takes every g-th m-tile,
// g being the number of CTAs that own the same n-tile.
// CTA pairs: both CTAs of a pair walk the pair's tiles; tm counts 256-row tiles.
template <bool WS, bool CTA2 = false>
__device__ __forceinline__ bool tile_at(const GemmParams& p, int i, int& tm, int& tn) {
  if (CTA2) {
    const int tile = (blockIdx.x >> 1) + i * (gridDim.x >> 1);
    tm = tile / p.tiles_n;
    tn = tile - tm * p.tiles_n;
    return tile < p.tiles_m * p.tiles_n;
  }
  if (WS) {
    tn = blockIdx.x % p.tiles_n;
    const int r = blockIdx.x / p.tiles_n;
    const int g = ((int)gridDim.x - 1 - tn) / p.tiles_n + 1;
    tm = r + i * g;
    return tm < p.tiles_m;
  }
  const int tile = blockIdx.x + i * gridDim.x;
  tm = tile / p.tiles_n;
  tn = tile - tm * p.tiles_n;
  return tile < p.tiles_m * p.tiles_n;
}

// RQ (CTA pairs, no GLU): the epilogue also quantizes the output rows for the next layer (Fig. 2 of
// the paper on u = what the plain epilogue writes): pass 1 is the plain epilogue, which also keeps
// the row maxima and writes u back over its accumulators; every thread then publishes the maximum
// of its row over its warp's columns as a tagged word, polls the words of the other column parts
// of the row (its own CTA's other warps and the other pairs of its group, which work on the same
// rows at the same time), and pass 2 turns u into codes.  The next tile's MMAs run meanwhile in
// the other accumulator buffer.  The pairs of a group (tiles_n consecutive pairs) always share
// their rows, so the grid is a multiple of tiles_n pairs.
template <int BN, int STAGES, int EW, bool WS, bool BPACK, int ACCK, bool DEBUG, bool CTA2 = false, bool RQ = false>
__global__ void __launch_bounds__(32 * (2 + EW), 1)
qgemm_i8_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_r, const GemmParams p) {
  using Cfg = GemmCfg<BN, STAGES, EW, WS, CTA2>;
  constexpr int HALF = BN / 2;
  constexpr int SBUFS = Cfg::kStageBufs;
  constexpr int TILE_M = CTA2 ? 2 * kBM : kBM;  // rows of a tile (of the pair's tile)
  static_assert(!BPACK || WS, "packed weights are unpacked into the resident slab");
  constexpr bool TF32 = (ACCK == kAccFloat);  // float operands: no activation scale, accumulators are binary32
  static_assert(!(TF32 && (BPACK || DEBUG)), "the float kind reads expanded weights and has no integer accumulators to dump");
  static_assert(!(TF32 && BN == 512), "512-column tiles exist for the 8-bit kind only");
  static_assert(!RQ || (CTA2 && !TF32 && !DEBUG && !WS), "the row-quantizing epilogue belongs to the 8-bit CTA-pair kernel");
  const uint32_t pair_rank = CTA2 ? cluster_ctarank() : 0u;  // 0 = leader: issues the MMAs, owns the barriers the pair shares
  const int row_in_tile = (int)pair_rank * kBM;               // this CTA's first row inside the tile

  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[STAGES];
  __shared__ uint64_t empty_bar[STAGES];
  __shared__ uint64_t tmem_full_bar[2];
  __shared__ uint64_t tmem_empty_bar[2];
  __shared__ uint64_t res_bar[EW][SBUFS];  // residual tile landed in a warp's staging buffer
  __shared__ uint64_t b_loaded_bar;        // WS: the CTA's weight slab (or its packed form) has landed
  __shared__ uint64_t b_ready_bar;         // WS + BPACK: every epilogue warp has unpacked its share
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
  const uint32_t smem_ring = smem_base;
  const uint32_t smem_res_b = smem_ring + STAGES * Cfg::kStageBytes;  // WS: resident weights, one 128-byte k-block after another
  const uint32_t smem_epi = smem_res_b + Cfg::kResidentBytes;
  const uint32_t smem_scale = smem_epi + Cfg::kEpiBytes;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint64_t t_start = global_timer_ns();
  const bool glu = (p.act == AQT_ACT_GLU) || (p.act == AQT_ACT_GLU_SWISH);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b);
    tma_prefetch_desc(&tm_y);
    if (p.residual != nullptr) tma_prefetch_desc(&tm_r);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&tmem_full_bar[b]), 1);
      mbar_init(smem_u32(&tmem_empty_bar[b]), CTA2 ? 2 * EW : EW);  // pair: both CTAs' epilogue warps release the leader's MMA
    }
    for (int w = 0; w < EW; ++w)
      for (int b = 0; b < SBUFS; ++b) mbar_init(smem_u32(&res_bar[w][b]), 1);
    mbar_init(smem_u32(&b_loaded_bar), 1);
    mbar_init(smem_u32(&b_ready_bar), EW);
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    if (CTA2) {
      tmem_alloc_pair(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
      tmem_relinquish();
    }
  }
  // everything above touched only this CTA's own state; from here on global memory is read
  grid_dependency_wait();
  // RQ: tag of this execution's exchange words (the call's tag mixed with the group's generation
  // counter, which the group's first CTA bumps when it has finished: a replayed graph repeats the call's tag)
  const int rq_group = RQ ? (int)(blockIdx.x >> 1) / p.tiles_n : 0;
  const uint32_t rq_tag = RQ ? mix_tag(p.tag, __ldcg(p.generation + rq_group)) : 0u;
  if (WS) {
    // scales and biases of the CTA's n-tile, once: values first, then (GLU) gates
    const int tn = blockIdx.x % p.tiles_n;
    for (int t = threadIdx.x; t < BN; t += blockDim.x) {
      int n, limit;
      if (glu) {
        n = (t < HALF) ? tn * HALF + t : p.N / 2 + tn * HALF + (t - HALF);
        limit = (t < HALF) ? p.N / 2 : p.N;
      } else {
        n = tn * BN + t;
        limit = p.N;
      }
      float wv = 0.0f, bv = 0.0f;
      if (n < limit) {
        wv = __ldg(p.s_w + n);
        if (p.bias != nullptr) bv = __ldg(p.bias + n);
      }
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_scale + t * 4), "f"(wv) : "memory");
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_scale + (BN + t) * 4), "f"(bv) : "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CTA2) cluster_sync_all();  // the peer's barriers are initialised before anything is signalled on them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      if (WS) {
        // the CTA's weight slab, once: int8 codes straight into the resident slab, or the packed
        // nibbles into the (still unused) epilogue staging area for the warps to unpack
        const int tn = blockIdx.x % p.tiles_n;
        const int row0 = glu ? tn * HALF : tn * BN;
        const int row1 = glu ? p.N / 2 + tn * HALF : tn * BN + HALF;
        const uint32_t bar = smem_u32(&b_loaded_bar);
        if (BPACK) {
          mbar_arrive_expect_tx(bar, (uint32_t)p.k_blocks * BN * 64);
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            tma_load_2d(smem_epi + kb * BN * 64, &tm_b, kb * 64, row0, bar);
            tma_load_2d(smem_epi + kb * BN * 64 + HALF * 64, &tm_b, kb * 64, row1, bar);
          }
        } else {
          mbar_arrive_expect_tx(bar, (uint32_t)p.k_blocks * Cfg::kBBytes);
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            tma_load_2d(smem_res_b + kb * Cfg::kBBytes, &tm_b, kb * kBK, row0, bar);
            tma_load_2d(smem_res_b + kb * Cfg::kBBytes + HALF * kBK, &tm_b, kb * kBK, row1, bar);
          }
        }
      }
      int tm, tn;
      for (int i = 0; ok && tile_at<WS, CTA2>(p, i, tm, tn); ++i) {
        // B rows of the two half-tiles: adjacent output channels, or (value, gate) halves for GLU
        const int row0 = glu ? tn * HALF : tn * BN;
        const int row1 = glu ? p.N / 2 + tn * HALF : tn * BN + HALF;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1, &abort_flag, t_start)) { ok = false; break; }
          const uint32_t bar = smem_u32(&full_bar[s]);
          const uint32_t stage = smem_ring + s * Cfg::kStageBytes;
          if (CTA2) {
            // The leader's barrier counts both CTAs' bytes; each CTA loads its 128 rows of A and
            // its half of the weight rows (leader: first half / values, peer: second half / gates).
            if (pair_rank == 0) mbar_arrive_expect_tx(bar, 2 * Cfg::kStageBytes);
            tma_load_2d_pair(stage, &tm_a, kb * kBK, tm * TILE_M + row_in_tile, bar);
            if (BN == 512) {
              // two MMAs of 256 columns per k-step: this CTA supplies 128 weight rows to each
              const int r = tn * BN + (int)pair_rank * 128;
              tma_load_2d_pair(stage + Cfg::kABytes, &tm_b, kb * kBK, r, bar);
              tma_load_2d_pair(stage + Cfg::kABytes + 128 * kBK, &tm_b, kb * kBK, r + 256, bar);
            } else {
              tma_load_2d_pair(stage + Cfg::kABytes, &tm_b, kb * kBK, pair_rank == 0 ? row0 : row1, bar);
            }
            continue;
          }
          mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
          tma_load_2d(stage, &tm_a, kb * kBK, tm * kBM, bar);
          if (!WS) {
            const int b_batch = p.batch_tiles_m > 0 ? (tm / p.batch_tiles_m) * p.batch_b_rows : 0;  // this batch's rows of B
            tma_load_2d(stage + Cfg::kABytes, &tm_b, kb * kBK, row0 + b_batch, bar);
            tma_load_2d(stage + Cfg::kABytes + HALF * kBK, &tm_b, kb * kBK, row1 + b_batch, bar);
          }
        }
      }
      grid_dependents_launch();  // every load of this CTA has been issued: the next kernel may be scheduled behind it
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && pair_rank == 0) {
      constexpr uint32_t idesc = TF32 ? idesc_tf32(Cfg::kMmaN, TILE_M) : idesc_i8(Cfg::kMmaN, TILE_M);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      if (WS) ok = mbar_wait(smem_u32(BPACK ? &b_ready_bar : &b_loaded_bar), 0, &abort_flag, t_start);
      int tm, tn;
      for (int i = 0; ok && tile_at<WS, CTA2>(p, i, tm, tn); ++i, ++tcount) {
        const uint32_t buf = tcount % Cfg::kAccBufs, aph = (tcount / Cfg::kAccBufs) & 1;
        if (!mbar_wait(smem_u32(&tmem_empty_bar[buf]), aph ^ 1, &abort_flag, t_start)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!mbar_wait(smem_u32(&full_bar[s]), ph, &abort_flag, t_start)) { ok = false; break; }
          tc_fence_after();
          const uint32_t stage = smem_ring + s * Cfg::kStageBytes;
          const uint64_t a_desc = smem_desc_k_major_sw128(stage);
          const uint64_t b_desc = smem_desc_k_major_sw128(WS ? smem_res_b + kb * Cfg::kBBytes : stage + Cfg::kABytes);
#pragma unroll
          for (int kk = 0; kk < kBK / kMmaK; ++kk) {
            // advancing K inside the 128-byte swizzle row: +32 bytes = +2 in the 16-byte address field
            const uint32_t accumulate = (kb | kk) != 0 ? 1u : 0u;
            if (TF32) {
              if (CTA2) tc_mma_tf32_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, accumulate);
              else tc_mma_tf32(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, accumulate);
            } else {
              if (CTA2) tc_mma_i8_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, accumulate);
              else tc_mma_i8(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, accumulate);
              if (BN == 512)  // columns 256 .. 511: the second 128 weight rows of each CTA's stage (16 KB further on)
                tc_mma_i8_pair(d_tmem + 256, a_desc + 2 * kk, b_desc + (128 * kBK >> 4) + 2 * kk, idesc, accumulate);
            }
          }
          // stage reusable (in both CTAs of a pair) once these MMAs have read it
          if (CTA2) tc_commit_pair(smem_u32(&empty_bar[s]));
          else tc_commit(smem_u32(&empty_bar[s]));
        }
        if (ok) {  // accumulator complete (in both CTAs' TMEM)
          if (CTA2) tc_commit_pair(smem_u32(&tmem_full_bar[buf]));
          else tc_commit(smem_u32(&tmem_full_bar[buf]));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int ew = warp - 2;
    const int quad = warp & 3;  // TMEM lane quadrant this warp may read
    const int chalf = ew >> 2;  // which share of the tile's output columns (0 .. EW/4 - 1)
    const uint32_t my_stage = smem_epi + ew * SBUFS * kStageBufBytes;
    const int out_cols_tile = glu ? HALF : BN;         // output columns per tile
    const int chunks = out_cols_tile / 32 / (EW / 4);  // 32-column chunks per epilogue warp and tile
    const bool has_res = p.residual != nullptr;
    const int n_value_limit = glu ? p.N / 2 : p.N;
    // where the scales of this warp's chunk c start: per-CTA slab (WS) or per-warp slab
    const uint32_t slab_sw = WS ? smem_scale + (uint32_t)(chalf * chunks * 32) * 4 : smem_scale + ew * 2 * Cfg::kSlabFloats * 4;
    const uint32_t slab_bias = WS ? slab_sw + BN * 4 : slab_sw + Cfg::kSlabFloats * 4;
    const uint32_t slab_chunk_stride = (WS || !glu) ? 128 : 256;  // bytes between consecutive chunks of this warp
    const uint32_t slab_gate_off = WS ? HALF * 4 : 128;           // gate columns relative to the value columns
    uint32_t store_count = 0;
    bool ok = true;
    const bool do_store = !RQ || p.has_y != 0;  // the fp32 output is written (always, without RQ)

    if (WS && BPACK) {
      // Sign-extend the CTA's packed weights into the resident slab, in the layout a swizzled
      // TMA load of int8 codes would have produced: row r of a k-block is 128 bytes, its 16-byte
      // chunk j sits at position j ^ (r & 7).  Exact (integers), done once per CTA.
      ok = mbar_wait(smem_u32(&b_loaded_bar), 0, &abort_flag, t_start);
      if (ok) {
        const int pieces = p.k_blocks * BN * 4;  // 16 packed bytes -> 32 codes each
        for (int q = (ew * 32 + lane); q < pieces; q += EW * 32) {
          const int kb = q / (BN * 4), rem = q - kb * (BN * 4);
          const int r = rem >> 2, piece = rem & 3;
          uint32_t w0, w1, w2, w3;
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                       : "r"(smem_epi + kb * BN * 64 + r * 64 + piece * 16)
                       : "memory");
          uint32_t o[8];
          unpack_word(w0, o[0], o[1]);
          unpack_word(w1, o[2], o[3]);
          unpack_word(w2, o[4], o[5]);
          unpack_word(w3, o[6], o[7]);
          const uint32_t row_base = smem_res_b + kb * Cfg::kBBytes + r * 128;
          const uint32_t d0 = row_base + (((2 * piece) ^ (r & 7)) << 4);
          const uint32_t d1 = row_base + (((2 * piece + 1) ^ (r & 7)) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(d0), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(d1), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        }
        fence_proxy_async_smem();  // the tensor core reads the slab through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&b_ready_bar));
        // nobody may overwrite the packed bytes (they sit in the staging buffers) before all have read them
        ok = mbar_wait(smem_u32(&b_ready_bar), 0, &abort_flag, t_start);
      }
    }

    int tm, tn;
    // residual prefetch for the very first chunk of this warp
    if (ok && has_res && lane == 0 && tile_at<WS, CTA2>(p, 0, tm, tn)) {
      const int oc0 = tn * out_cols_tile + chalf * chunks * 32, r0 = tm * TILE_M + row_in_tile + quad * 32;
      const uint32_t bar = smem_u32(&res_bar[ew][0]);
      mbar_arrive_expect_tx(bar, kStageBufBytes);
      tma_load_2d(my_stage, &tm_r, oc0 < p.n_out ? oc0 : 0, r0 < p.M ? r0 : 0, bar);
    }

    for (int i = 0; ok && tile_at<WS, CTA2>(p, i, tm, tn); ++i) {
      const uint32_t buf = i % Cfg::kAccBufs, aph = (i / Cfg::kAccBufs) & 1;
      const int out0 = tn * out_cols_tile;  // first output column of the tile
      const int row0_warp = tm * TILE_M + row_in_tile + quad * 32;  // first output row of this warp
      const int m = row0_warp + lane;
      const bool row_ok = m < p.M;

      if (!WS && Cfg::kScaleSlab) {
        // this warp's s_w / bias slices for the tile -> shared memory (before the accumulator is ready)
        __syncwarp();
        for (int c = 0; c < chunks; ++c) {
          const int col = (chalf * chunks + c) * 32;
          const int nv = (glu ? out0 : tn * BN) + col + lane;  // value channel of this lane
          const uint32_t off = c * slab_chunk_stride + lane * 4;
          float wv = 0.0f, bv = 0.0f;
          if (nv < n_value_limit) {
            wv = __ldg(p.s_w + nv);
            if (p.bias != nullptr) bv = __ldg(p.bias + nv);
          }
          asm volatile("st.shared.f32 [%0], %1;" ::"r"(slab_sw + off), "f"(wv) : "memory");
          asm volatile("st.shared.f32 [%0], %1;" ::"r"(slab_bias + off), "f"(bv) : "memory");
          if (glu) {
            const int ng = p.N / 2 + out0 + col + lane;  // gate channel
            float wg = 0.0f, bg = 0.0f;
            if (ng < p.N) {
              wg = __ldg(p.s_w + ng);
              if (p.bias != nullptr) bg = __ldg(p.bias + ng);
            }
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(slab_sw + off + slab_gate_off), "f"(wg) : "memory");
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(slab_bias + off + slab_gate_off), "f"(bg) : "memory");
          }
        }
      }
      const float sx = TF32 ? 1.0f : ((p.s_x_kind == AQT_SCALE_ROW) ? (row_ok ? __ldg(p.s_x + m) : 0.0f) : __ldg(p.s_x));
      float rq_amax = 0.0f;  // RQ: maximum of this thread's row over this warp's columns
      __syncwarp();

      if (!mbar_wait(smem_u32(&tmem_full_bar[buf]), aph, &abort_flag, t_start)) break;
      tc_fence_after();
      const uint32_t lane_addr = tmem_base + buf * BN + ((uint32_t)(quad * 32) << 16);

      for (int c = 0; c < chunks; ++c) {
        const int col = (chalf * chunks + c) * 32;  // column offset inside the tile's output
        const int oc = out0 + col;                  // first global output column of this chunk
        const uint32_t sb = store_count % SBUFS;
        const uint32_t sbuf = my_stage + sb * kStageBufBytes;
        const uint32_t c_sw = slab_sw + c * slab_chunk_stride, c_bias = slab_bias + c * slab_chunk_stride;
        float a[32];
        uint32_t acc[32];
        const bool last_chunk = (c == chunks - 1);
        if (!glu) {
          tmem_ld_32x32(lane_addr + col, acc);
          tmem_ld_wait();
          if (last_chunk && !RQ) {
            // accumulator buffer read out by this warp: hand it back before the arithmetic
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (CTA2) mbar_arrive_cluster(smem_u32(&tmem_empty_bar[buf]), 0);
              else mbar_arrive(smem_u32(&tmem_empty_bar[buf]));
            }
          }
          if (DEBUG) {
            if (p.acc_debug != nullptr && row_ok) {
              const int n0 = tn * BN + col;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (n0 + j < p.N) p.acc_debug[(int64_t)m * p.N + n0 + j] = (int32_t)acc[j];
            }
          }
          if (Cfg::kScaleSlab) dequant32<ACCK>(acc, sx, c_sw, c_bias, a);
          else dequant32_gmem<ACCK>(acc, sx, p.s_w, p.bias, tn * BN + col, p.N, a);
          if (p.act == AQT_ACT_SWISH) swish32(a);
        } else {
          // gates first: g = sigmoid(z_gate); then the values are scaled by it
          float g[32];
          tmem_ld_32x32(lane_addr + HALF + col, acc);
          tmem_ld_wait();
          if (DEBUG) {
            if (p.acc_debug != nullptr && row_ok) {
              const int ng = p.N / 2 + oc;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (ng + j < p.N) p.acc_debug[(int64_t)m * p.N + ng + j] = (int32_t)acc[j];
            }
          }
          if (Cfg::kScaleSlab) dequant32<ACCK>(acc, sx, c_sw + slab_gate_off, c_bias + slab_gate_off, g);
          else dequant32_gmem<ACCK>(acc, sx, p.s_w, p.bias, p.N / 2 + oc, p.N, g);
#pragma unroll
          for (int j = 0; j < 32; ++j) g[j] = sigmoid_f(g[j]);
          tmem_ld_32x32(lane_addr + col, acc);
          tmem_ld_wait();
          if (last_chunk) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (CTA2) mbar_arrive_cluster(smem_u32(&tmem_empty_bar[buf]), 0);
              else mbar_arrive(smem_u32(&tmem_empty_bar[buf]));
            }
          }
          if (DEBUG) {
            if (p.acc_debug != nullptr && row_ok) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (oc + j < p.N / 2) p.acc_debug[(int64_t)m * p.N + oc + j] = (int32_t)acc[j];
            }
          }
          if (Cfg::kScaleSlab) dequant32<ACCK>(acc, sx, c_sw, c_bias, a);
          else dequant32_gmem<ACCK>(acc, sx, p.s_w, p.bias, oc, p.N / 2, a);
#pragma unroll
          for (int j = 0; j < 32; ++j) a[j] = a[j] * g[j];
          if (p.act == AQT_ACT_GLU_SWISH) swish32(a);
        }

        // the chunk this warp handles after this one (for the residual prefetch)
        int ntm = tm, ntn = tn, nc = c + 1;
        bool have_next = true;
        if (nc == chunks) {
          nc = 0;
          have_next = tile_at<WS, CTA2>(p, i + 1, ntm, ntn);
        }
        const int noc = ntn * out_cols_tile + (chalf * chunks + nc) * 32, nr = ntm * TILE_M + row_in_tile + quad * 32;

        if (has_res) {
          if (SBUFS == 2) {
            // Buffers alternate: the residual of this chunk was requested one chunk ago into `sb`.
            // Request the next chunk's residual into the other buffer once the store that last
            // used it has been read out, then wait for this chunk's tile.
            if (lane == 0) {
              tma_store_wait_read<0>();
              if (have_next) {
                const uint32_t nb = (store_count + 1) % SBUFS;
                const uint32_t bar = smem_u32(&res_bar[ew][nb]);
                mbar_arrive_expect_tx(bar, kStageBufBytes);
                // a box that would start outside the tensor is redirected to its origin (never read)
                tma_load_2d(my_stage + nb * kStageBufBytes, &tm_r, noc < p.n_out ? noc : 0, nr < p.M ? nr : 0, bar);
              }
            }
            __syncwarp();
          }
          if (!mbar_wait(smem_u32(&res_bar[ew][sb]), (store_count / SBUFS) & 1, &abort_flag, t_start)) { ok = false; break; }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t src = sbuf + lane * 128 + ((j ^ (lane & 7)) << 4);
            float r0, r1, r2, r3;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r0), "=f"(r1), "=f"(r2), "=f"(r3) : "r"(src) : "memory");
            a[4 * j + 0] = __fmaf_rn(p.residual_scale, a[4 * j + 0], r0);
            a[4 * j + 1] = __fmaf_rn(p.residual_scale, a[4 * j + 1], r1);
            a[4 * j + 2] = __fmaf_rn(p.residual_scale, a[4 * j + 2], r2);
            a[4 * j + 3] = __fmaf_rn(p.residual_scale, a[4 * j + 3], r3);
          }
          __syncwarp();  // every lane has read its residual row before the buffer is overwritten
        } else if (do_store) {
          // staging buffer free once the bulk store that last used it has been read out
          if (lane == 0) tma_store_wait_read<SBUFS - 1>();
          __syncwarp();
        }
        if constexpr (RQ) {
          // u stays in tensor memory, over the accumulators it was made from, until the row's scale is known
          float cmax = 0.0f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            cmax = fmaxf(cmax, fabsf(a[j]));
            acc[j] = __float_as_uint(a[j]);
          }
          if (oc < p.n_out) rq_amax = fmaxf(rq_amax, cmax);  // columns beyond N contribute nothing
          tmem_st_32x32(lane_addr + col, acc);
        }
        // row `lane` of the 32 x 32 box; 16-byte chunk j sits at (j ^ (row & 7)) under the 128-byte swizzle
        if (do_store) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t dst = sbuf + lane * 128 + ((j ^ (lane & 7)) << 4);
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(a[4 * j]), "f"(a[4 * j + 1]),
                         "f"(a[4 * j + 2]), "f"(a[4 * j + 3])
                         : "memory");
          }
          fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0 && do_store) {
          // boxes that start inside the output are clipped at its edges by the copy engine
          if (oc < p.n_out && row0_warp < p.M) tma_store_2d(&tm_y, sbuf, oc, row0_warp);
          tma_store_commit();
          if (has_res && SBUFS == 1) {
            // single buffer: the next chunk's residual can only be requested once this store has
            // read the buffer out (the warp is otherwise idle until its next chunk)
            tma_store_wait_read<0>();
            if (have_next) {
              const uint32_t bar = smem_u32(&res_bar[ew][0]);
              mbar_arrive_expect_tx(bar, kStageBufBytes);
              tma_load_2d(my_stage, &tm_r, noc < p.n_out ? noc : 0, nr < p.M ? nr : 0, bar);
            }
          }
        }
        ++store_count;
      }
      if (!ok) break;
      if constexpr (RQ) {
        // ---------------------------------------------------------- the row's maximum over all of N
        const int parts = p.exchange_parts;
        const int my_part = tn * (EW / 4) + chalf;
        uint64_t* xrow = p.exchange + (size_t)m * parts;  // rows up to the padded tile height are allocated
        st_relaxed_gpu_64(xrow + my_part, ((uint64_t)rq_tag << 32) | __float_as_uint(rq_amax));
        uint32_t amax_bits = 0u;
        for (uint32_t spin = 1;; ++spin) {
          bool all = true;
          amax_bits = 0u;
          for (int q = 0; q < parts; q += 2) {  // parts is even: a pair has at least two column parts
            const ulonglong2 w = ld_relaxed_gpu_2x64(xrow + q);
            all = all && (uint32_t)(w.x >> 32) == rq_tag && (uint32_t)(w.y >> 32) == rq_tag;
            amax_bits = max(amax_bits, max((uint32_t)w.x, (uint32_t)w.y));
          }
          if (__all_sync(0xffffffffu, all)) break;
          if ((spin & 0x3F) == 0) {
            bool go_on = *(volatile int*)&abort_flag == 0;
            if (go_on && global_timer_ns() - t_start > kWaitLimitNs) {
              *(volatile int*)&abort_flag = 1;
              atomicExch(&g_device_status, AQT_ERR_TIMEOUT);
              go_on = false;
            }
            if (!__all_sync(0xffffffffu, go_on)) { ok = false; break; }
          }
        }
        if (!ok) break;
        // ---------------------------------------------------------- pass 2: scale, codes
        const ScaleCtx sc = make_scale_ctx(__uint_as_float(amax_bits), p.qmax_out);
        if (my_part == 0 && row_ok) p.s_out[m] = sc.s;
        tmem_st_wait();  // this warp's stores of pass 1
        for (int c = 0; c < chunks; ++c) {
          const int col = (chalf * chunks + c) * 32;
          const int oc = out0 + col;
          uint32_t u[32], w[8];
          tmem_ld_32x32(lane_addr + col, u);
          tmem_ld_wait();
          if (c == chunks - 1) {
            // the tile has been read out by this warp: the accumulator buffer goes back to the MMA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(smem_u32(&tmem_empty_bar[buf]), 0);
          }
          if (p.rounding == AQT_ROUND_HALF_UP_FLOOR) codes_of<AQT_ROUND_HALF_UP_FLOOR, false, 32>(u, sc, p.qmax_out, w);
          else codes_of<AQT_ROUND_NEAREST_EVEN, false, 32>(u, sc, p.qmax_out, w);
          if (row_ok && oc < p.n_out) {
            uint4* dst = reinterpret_cast<uint4*>(p.q_out + (size_t)m * p.n_out + oc);
            dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            if (oc + 16 < p.n_out) dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
      }
    }
    if (lane == 0) tma_store_wait_all();
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (abort_flag && threadIdx.x == 0) {
    // give bulk copies that were in flight when a wait gave up time to land before smem is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) {
    }
  }
  __syncthreads();
  if (CTA2) cluster_sync_all();  // neither CTA leaves (or frees TMEM) while its peer may still signal it or use its memory
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (CTA2) tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
    else tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
  if (RQ) {
    // every CTA of the group has read the counter long since (this one could not finish its tiles without them)
    if (threadIdx.x == 0 && blockIdx.x == (unsigned)(2 * rq_group * p.tiles_n)) p.generation[rq_group] = __ldcg(p.generation + rq_group) + 1u;
  }
}

// Self-test of the bounded wait: one CTA waits on an mbarrier that nothing ever arrives on, with
// a short limit.  The wait must give up, record AQT_ERR_TIMEOUT in the device status word and let
// the kernel return normally (the context stays usable).
__global__ void bounded_wait_selftest_kernel(uint64_t limit_ns, int* gave_up) {
  __shared__ uint64_t never_signalled;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&never_signalled), 1);
    fence_barrier_init();
  }
  __syncthreads();
  const bool ok = mbar_wait(smem_u32(&never_signalled), 0, &abort_flag, global_timer_ns(), limit_ns);
  __syncthreads();
  if (threadIdx.x == 0) *gave_up = ok ? 0 : 1;
}

// ------------------------------------------------------------------------------------------------
// Host side: tensor maps and launch

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// 2-D row-major tensor [rows, cols] with `pitch_bytes` between rows; box [box_rows, box_cols];
// swizzle_bytes: 128 or 32 (box_cols * element size must then be that many bytes), or 0 for none.
static int make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t rows, uint64_t cols,
                       uint64_t pitch_bytes, uint32_t box_rows, uint32_t box_cols, int swizzle_bytes = 128) {
  EncodeTiledFn enc = get_encode_tiled();
  if (enc == nullptr) {
    if (debug_enabled()) fprintf(stderr, "[aqt] driver entry point for tensor map encoding not found\n");
    return AQT_ERR_CUDA;
  }
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE),
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS && debug_enabled())
    fprintf(stderr, "[aqt] tensor map encode failed: CUresult %d (rows %llu cols %llu pitch %llu box %u x %u base %p)\n", (int)r,
            (unsigned long long)rows, (unsigned long long)cols, (unsigned long long)pitch_bytes, box_rows, box_cols, base);
  return r == CUDA_SUCCESS ? AQT_OK : AQT_ERR_CUDA;
}

// Rounds of a persistent grid over the tiles: fewer rounds of fuller waves win.
static int pick_bn(int64_t M, int64_t N, bool glu, int sms) {
  const int64_t tiles_m = ceil_div(M, kBM);
  int best_bn = 128;
  double best_cost = 1e300;
  const int cands[3] = {256, 128, 64};
  for (int i = 0; i < 3; ++i) {
    const int bn = cands[i];
    if (glu && bn == 64) continue;  // a GLU tile needs 32 value + 32 gate columns per epilogue warp pair
    const int64_t tiles = tiles_m * ceil_div(N, bn);
    const int64_t rounds = ceil_div(tiles, sms);
    // per-tile cost: proportional to BN, plus a fixed per-tile overhead worth ~24 columns
    const double cost = (double)rounds * (bn + 24);
    if (cost < best_cost) {
      best_cost = cost;
      best_bn = bn;
    }
  }
  return best_bn;
}

// b: weight codes as the kernel reads them -- int8 [N, K], or (BPACK) packed nibbles [N, K/2].
template <int BN, int STAGES, int EW, bool WS, bool BPACK, int ACCK, bool DEBUG, bool CTA2 = false, bool RQ = false>
static int launch_qgemm_inst(const int8_t* a, const void* b, float* y, int64_t ldy, const GemmParams& p0, cudaStream_t st) {
  using Cfg = GemmCfg<BN, STAGES, EW, WS, CTA2>;
  GemmParams p = p0;
  p.tiles_m = (int)ceil_div(p.M, CTA2 ? 2 * kBM : kBM);
  p.tiles_n = (int)ceil_div(p.N, BN);
  p.k_blocks = (int)ceil_div(p.K, kBK);
  const int sms = sm_count();
  if (sms <= 0) return AQT_ERR_CUDA;
  {
    const bool glu = (p.act == AQT_ACT_GLU) || (p.act == AQT_ACT_GLU_SWISH);
    if ((glu ? BN / 2 : BN) / 32 / (EW / 4) < 1) return AQT_ERR_UNSUPPORTED;  // a warp without columns would never release TMEM
    if (WS && (p.k_blocks > kWsMaxKBlocks || p.tiles_n > sms)) return AQT_ERR_UNSUPPORTED;
    if (BN == 512 && glu) return AQT_ERR_UNSUPPORTED;  // value and gate halves are not laid out for two MMAs per step
    if (CTA2 && p.M <= kBM) return AQT_ERR_UNSUPPORTED;
  }
  CUtensorMap tm_a, tm_b, tm_y, tm_r;
  int rc = make_map_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, a, (uint64_t)p.M, (uint64_t)p.K,
                       (uint64_t)(p.a_pitch != 0 ? p.a_pitch : p.K), kBM, kBK);
  if (rc != AQT_OK) return rc;
  if (BPACK) {
    rc = make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b, (uint64_t)p.N, (uint64_t)p.K / 2, (uint64_t)p.K / 2, BN / 2, 64, 0);
  } else {
    rc = make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b, (uint64_t)(p.b_rows != 0 ? p.b_rows : p.N), (uint64_t)p.K, (uint64_t)p.K,
                     BN == 512 ? 128 : BN / 2, kBK);
  }
  if (rc != AQT_OK) return rc;
  if (p.batch_tiles_m > 0 && (WS || CTA2)) return AQT_ERR_UNSUPPORTED;
  if (RQ && !p.has_y) {
    tm_y = tm_a;  // never dereferenced
  } else {
    rc = make_map_2d(&tm_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, y, (uint64_t)p.M, (uint64_t)p.n_out, (uint64_t)ldy * 4, kStoreBoxRows,
                     kStoreBoxCols);
    if (rc != AQT_OK) return rc;
  }
  if (p.residual != nullptr) {
    rc = make_map_2d(&tm_r, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, p.residual, (uint64_t)p.M, (uint64_t)p.n_out, (uint64_t)p.ldr * 4,
                     kStoreBoxRows, kStoreBoxCols);
    if (rc != AQT_OK) return rc;
  } else {
    tm_r = tm_y;  // never dereferenced
  }
  auto kernel = qgemm_i8_kernel<BN, STAGES, EW, WS, BPACK, ACCK, DEBUG, CTA2, RQ>;
  static std::atomic<uint64_t> smem_opted_in{0};
  rc = ensure_dynamic_smem(kernel, Cfg::kSmemBytes, smem_opted_in);
  if (rc != AQT_OK) return rc;
  const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
  unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  if (WS && (int)grid < p.tiles_n) grid = (unsigned)p.tiles_n;  // every n-tile needs an owner
  if (CTA2) {
    // one cluster of two CTAs per tile in flight
    int64_t pairs = sms / 2;
    if (RQ) {
      // the pairs that share rows (tiles_n consecutive ones) wait on one another: whole groups only,
      // every one of them on an SM of its own
      if (p.tiles_n > pairs || p.exchange_parts != p.tiles_n * (EW / 4) || p.exchange_parts % 2 != 0) return AQT_ERR_UNSUPPORTED;
      pairs = pairs / p.tiles_n * p.tiles_n;
    }
    grid = 2u * (unsigned)(tiles < pairs ? tiles : pairs);
    return launch_pdl(kernel, dim3(grid, 1, 1), dim3(Cfg::kThreads, 1, 1), Cfg::kSmemBytes, st, 2, tm_a, tm_b, tm_y, tm_r, p);
  }
  return launch_pdl(kernel, dim3(grid, 1, 1), dim3(Cfg::kThreads, 1, 1), Cfg::kSmemBytes, st, 1, tm_a, tm_b, tm_y, tm_r, p);
}

template <int BN, int STAGES, int EW, bool WS, bool BPACK, bool CTA2 = false>
static int launch_qgemm_cfg(const int8_t* a, const void* b, float* y, int64_t ldy, const GemmParams& p, cudaStream_t st) {
  if (p.kind == 1) {
    if constexpr (!BPACK && BN != 512) {
      if (p.acc_debug == nullptr) return launch_qgemm_inst<BN, STAGES, EW, WS, false, kAccFloat, false, CTA2>(a, b, y, ldy, p, st);
    }
    return AQT_ERR_UNSUPPORTED;
  }
  if (p.acc_debug != nullptr) return launch_qgemm_inst<BN, STAGES, EW, WS, BPACK, kAccInt32, true, CTA2>(a, b, y, ldy, p, st);
  if (p.small_acc) return launch_qgemm_inst<BN, STAGES, EW, WS, BPACK, kAccInt32Small, false, CTA2>(a, b, y, ldy, p, st);
  return launch_qgemm_inst<BN, STAGES, EW, WS, BPACK, kAccInt32, false, CTA2>(a, b, y, ldy, p, st);
}

// ------------------------------------------------------------------------------------------------
// Choice of the kernel configuration ("plan") for a shape, and the launch of a plan

// Every configuration of the kernel template that the library instantiates.
enum GemmPlan {
  kPlanNone = 0,
  kPlanWs128E16,        // weight stationary (K <= 512), 128-column tiles, sixteen epilogue warps
  kPlanWs128E8,         // the same with eight epilogue warps: the GLU forms (64 output columns per tile)
  kPlanStream256S3E16,  // both operands streamed, 256-column tiles, shallow K
  kPlanStream256S4E4,   //   deep K: four-warp epilogue, deeper ring
  kPlanStream256S4E8,   //   float kind
  kPlanStream128S4E16,
  kPlanStream128S6E4,
  kPlanStream128S4E8,   //   GLU at width 128
  kPlanStream64S5E8,
  kPlanStream64S8E4,
  kPlanPair256S4E8,     // CTA pairs on 256-row tiles
  kPlanPair256S6E4,
  kPlanPair128S6E8,
  kPlanPair128S8E4,
  kPlanPair512S3E16,    // CTA pairs on 256 x 512 tiles, one accumulator buffer (few, deep tiles)
  kPlanCount
};
static const char* const kGemmPlanNames[kPlanCount] = {
    "none",          "ws128e16",      "ws128e8",       "stream256s3e16", "stream256s4e4", "stream256s4e8",
    "stream128s4e16", "stream128s6e4", "stream128s4e8", "stream64s5e8",   "stream64s8e4",  "pair256s4e8",
    "pair256s6e4",   "pair128s6e8",   "pair128s8e4",   "pair512s3e16"};
static const char* gemm_plan_name(int plan) { return plan > 0 && plan < kPlanCount ? kGemmPlanNames[plan] : kGemmPlanNames[0]; }
static int gemm_plan_by_name(const char* name) {
  if (name == nullptr) return kPlanNone;
  for (int i = 1; i < kPlanCount; ++i)
    if (strcmp(name, kGemmPlanNames[i]) == 0) return i;
  return kPlanNone;
}

// What the choice depends on.  K in bytes of contraction per operand row (see GemmParams).
struct GemmShape {
  int64_t M, N, K;
  int act;
  int kind;      // 0: 8-bit codes, 1: float kind
  bool batched;  // stacked batches: streaming kernel, one CTA per tile
};

// True if the weight-stationary kernel takes this shape (and can therefore unpack 4-bit weights itself).
static bool qgemm_uses_ws(int64_t N, int64_t K, int sms) {
  if (tuning_env("AQT_NO_WS") != nullptr) return false;  // tuning builds: force the streaming kernel
  return ceil_div(K, kBK) <= kWsMaxKBlocks && ceil_div(N, 128) <= sms;
}

// sms: multiprocessors of the device the launch will go to.
static int plan_qgemm(const GemmShape& g, int sms) {
  const bool glu = (g.act == AQT_ACT_GLU) || (g.act == AQT_ACT_GLU_SWISH);
  const bool f32 = g.kind == 1;
  if (!g.batched && qgemm_uses_ws(g.N, g.K, sms)) return glu ? kPlanWs128E8 : kPlanWs128E16;  // a GLU tile has 64 output columns
  // "Deep" configuration (four-warp epilogue, longest ring): pays off when K is deep AND every
  // CTA walks many tiles; with few tiles per CTA the exposed epilogue of the last tile costs more
  // than the extra ring stages gain (measured at M = 12 800 .. 25 600).
  bool deep_k = g.K >= 2048 && !glu && ceil_div(g.M, kBM) * ceil_div(g.N, 256) >= 4 * sms;
  // Float kind: a k-block takes as many tensor-core clocks as an 8-bit one but holds a quarter of
  // the elements, so every shape is "deep" in bytes and the epilogue is a small part of a tile
  // unless it evaluates an activation (measured: the four-warp epilogue wins at 12 800 x 512 x
  // 2048 and 65 536 x 1024 x 4096 without activation, loses by 20-40 % with Swish).
  if (f32) deep_k = g.act == AQT_ACT_NONE && g.K >= 8192;
  if (const char* e = tuning_env("AQT_DEEP")) {
    if (!glu) deep_k = atoi(e) != 0;
  }
  const int pairs = sms / 2;
  // Pairs pay off only for deep K and at least two full rounds of pair tiles (measured: +4 % at
  // 65 536 x 1024 x 4096 with the deep configuration, +9 % at 25 600 x 512 x 2048 with the
  // eight-warp epilogue, no gain at M = 12 800 or at K = 1024); everything else takes one CTA per tile.
  // (the 8-bit kind's GLU shapes are faster on single CTAs; the float kind's gain 3 % on pairs)
  const bool two_rounds_of_pairs = (!glu || f32) && ceil_div(g.M, 2 * kBM) * ceil_div(g.N, 256) >= 2 * pairs;
  // (float kind, measured: pairs win 6-10 % at M >= 25 600, lose 10 % at 12 800 x 2048 x 512)
  bool pairs_ok = f32 ? (two_rounds_of_pairs && g.M >= 2 * kBM * pairs) : (deep_k || (g.K >= 2048 && two_rounds_of_pairs));
  if (tuning_env("AQT_NO_PAIRS") != nullptr) pairs_ok = false;
  if (tuning_env("AQT_FORCE_PAIRS") != nullptr) pairs_ok = true;
  if (!g.batched && g.M > kBM) {
    // Few, deep tiles (K >= 2048, all of N within one or two 512-column tiles, at most one round of
    // 256 x 512 tiles over the pairs): each pair takes one whole tile, so the activations are read
    // once, the weights once per 256 rows, and no SM waits for a second, mostly empty round.
    bool wide = !f32 && !glu && g.K >= 2048 && g.N % 512 == 0 && ceil_div(g.M, 2 * kBM) * (g.N / 512) <= pairs;
    if (const char* e = tuning_env("AQT_WIDE_PAIRS")) wide = !f32 && !glu && atoi(e) != 0;
    if (wide) return kPlanPair512S3E16;
  }
  if (!g.batched && pairs_ok && g.M > kBM) {
    // CTA pairs on 256-row tiles; width by the number of rounds over the pairs
    const int64_t tiles_m2 = ceil_div(g.M, 2 * kBM);
    const double cost256 = (double)ceil_div(tiles_m2 * ceil_div(g.N, 256), pairs) * (256 + 24);
    const double cost128 = (double)ceil_div(tiles_m2 * ceil_div(g.N, 128), pairs) * (128 + 24);
    int bn2 = cost256 <= cost128 ? 256 : 128;
    if (const char* e = tuning_env("AQT_BN")) {
      if (atoi(e) == 128 || atoi(e) == 256) bn2 = atoi(e);
    }
    // The four-warp epilogue / deeper ring pays off for pairs only from K = 4096 bytes (measured at
    // 65 536 x 1024 x 4096: 2753 vs 2671 TOPS burst, equal sustained; float kind 801 vs 752
    // TFLOP/s); at K = 2048 the eight-warp epilogue with four stages is 20-27 % faster (41.1 vs
    // 52.3 us at 37 888 x 512 x 2048, where the deep-K rule first applies; 83.1 vs 104.9 us at 65 536).
    bool dp = deep_k && g.K >= 4096;
    if (const char* e = tuning_env("AQT_DEEP_PAIRS")) dp = atoi(e) != 0;
    if (bn2 == 256) return dp ? kPlanPair256S6E4 : kPlanPair256S4E8;
    return dp ? kPlanPair128S8E4 : kPlanPair128S6E8;
  }
  int bn = pick_bn(g.M, g.N, glu, sms);
  // operand bytes per output are four times those of the 8-bit kind: the widest tile wins whenever it
  // still gives every SM a tile (a weight gradient has few, very deep tiles and takes narrow ones)
  if (f32 && g.N >= 256 && ceil_div(g.M, kBM) * ceil_div(g.N, 256) >= sms) bn = 256;
  if (const char* e = tuning_env("AQT_BN")) {
    const int v = atoi(e);
    if ((v == 64 && !glu) || v == 128 || v == 256) bn = v;
  }
  // Deep K: operand loads bound the tile, so the ring gets the shared memory and four warps run
  // the (short) epilogue.  Shallow K: the epilogue bounds the tile and gets more warps.
  // Float kind: a tile's MMA time is four times that of the 8-bit kind for the same epilogue, so
  // eight epilogue warps keep up and the shared memory they free buys the fourth ring stage
  // (measured 2-10 % faster than three stages / sixteen warps and than four stages / four warps:
  // 59.8 vs 62.4 us at 12 800 x 2048 x 512 Swish, 362 vs 398 us at 65 536 x 2048 x 1024 GLU).  The
  // 8-bit kind loses with it wherever the epilogue evaluates an activation or M is small.
  if (bn == 256 && f32) return kPlanStream256S4E8;
  if (bn == 256) return deep_k ? kPlanStream256S4E4 : kPlanStream256S3E16;
  // every epilogue warp needs at least one 32-column chunk: a GLU tile of width 128 has only
  // 64 output columns, i.e. two chunks per lane quadrant
  if (bn == 128 && glu) return kPlanStream128S4E8;
  if (bn == 128) return deep_k ? kPlanStream128S6E4 : kPlanStream128S4E16;
  return deep_k ? kPlanStream64S8E4 : kPlanStream64S5E8;
}

// Tile width and epilogue warps of each plan (same order as GemmPlan).
static const int kGemmPlanBn[kPlanCount] = {0, 128, 128, 256, 256, 256, 128, 128, 128, 64, 64, 256, 256, 128, 128, 512};
static const int kGemmPlanEw[kPlanCount] = {0, 16, 8, 16, 4, 8, 16, 4, 8, 8, 4, 8, 4, 8, 4, 16};

// True if `plan` can run this shape at all (used when a caller names the plan itself).
static bool gemm_plan_takes(int plan, const GemmShape& g, int sms) {
  if (plan <= kPlanNone || plan >= kPlanCount) return false;
  const bool glu = (g.act == AQT_ACT_GLU) || (g.act == AQT_ACT_GLU_SWISH);
  const bool ws = plan == kPlanWs128E16 || plan == kPlanWs128E8;
  const bool pair = plan >= kPlanPair256S4E8 && plan <= kPlanPair512S3E16;
  if (ws && (g.batched || ceil_div(g.K, kBK) > kWsMaxKBlocks || ceil_div(g.N, 128) > sms)) return false;
  if (pair && (g.batched || g.M <= kBM)) return false;
  if (plan == kPlanPair512S3E16 && (glu || g.kind != 0)) return false;
  // every epilogue warp needs at least one 32-column chunk of the tile's output columns
  const int out_cols = glu ? kGemmPlanBn[plan] / 2 : kGemmPlanBn[plan];
  return out_cols / 32 / (kGemmPlanEw[plan] / 4) >= 1;
}

// a: int8 [M, K] codes.  b: int8 [N, K] codes, or -- only if b_packed and a weight-stationary plan --
// packed nibbles [N, K/2].  All dense, 16-byte aligned.
static int launch_qgemm_plan(int plan, const int8_t* a, const void* b, bool b_packed, float* y, int64_t ldy, const GemmParams& p,
                             cudaStream_t st) {
  switch (plan) {
    case kPlanWs128E16:
      return b_packed ? launch_qgemm_cfg<128, 6, 16, true, true>(a, b, y, ldy, p, st) : launch_qgemm_cfg<128, 6, 16, true, false>(a, b, y, ldy, p, st);
    case kPlanWs128E8:
      return b_packed ? launch_qgemm_cfg<128, 6, 8, true, true>(a, b, y, ldy, p, st) : launch_qgemm_cfg<128, 6, 8, true, false>(a, b, y, ldy, p, st);
    default: break;
  }
  if (b_packed) return AQT_ERR_UNSUPPORTED;
  switch (plan) {
    case kPlanStream256S3E16: return launch_qgemm_cfg<256, 3, 16, false, false>(a, b, y, ldy, p, st);
    case kPlanStream256S4E4: return launch_qgemm_cfg<256, 4, 4, false, false>(a, b, y, ldy, p, st);
    case kPlanStream256S4E8: return launch_qgemm_cfg<256, 4, 8, false, false>(a, b, y, ldy, p, st);
    case kPlanStream128S4E16: return launch_qgemm_cfg<128, 4, 16, false, false>(a, b, y, ldy, p, st);
    case kPlanStream128S6E4: return launch_qgemm_cfg<128, 6, 4, false, false>(a, b, y, ldy, p, st);
    case kPlanStream128S4E8: return launch_qgemm_cfg<128, 4, 8, false, false>(a, b, y, ldy, p, st);
    case kPlanStream64S5E8: return launch_qgemm_cfg<64, 5, 8, false, false>(a, b, y, ldy, p, st);
    case kPlanStream64S8E4: return launch_qgemm_cfg<64, 8, 4, false, false>(a, b, y, ldy, p, st);
    case kPlanPair256S4E8: return launch_qgemm_cfg<256, 4, 8, false, false, true>(a, b, y, ldy, p, st);
    case kPlanPair256S6E4: return launch_qgemm_cfg<256, 6, 4, false, false, true>(a, b, y, ldy, p, st);
    case kPlanPair128S6E8: return launch_qgemm_cfg<128, 6, 8, false, false, true>(a, b, y, ldy, p, st);
    case kPlanPair128S8E4: return launch_qgemm_cfg<128, 8, 4, false, false, true>(a, b, y, ldy, p, st);
    case kPlanPair512S3E16: return launch_qgemm_cfg<512, 3, 16, false, false, true>(a, b, y, ldy, p, st);
    default: return AQT_ERR_UNSUPPORTED;
  }
}

// The CTA-pair configurations with the row-quantizing epilogue.  p carries q_out, s_out, the
// exchange area, tag, qmax_out, rounding, has_y; exchange_parts is filled in here.
static int rowquant_plan(int64_t M, int64_t N, int64_t K, int sms) {
  // Eight epilogue warps on 256 x 256 pair tiles throughout: both passes of a tile have to fit into
  // the next tile's MMA time (measured at 65 536 x 4096 -> 1024 with the fp32 output: 274 us against
  // 306 us with the four-warp epilogue and 288 us for matmul + row quantizer; 256 x 512 tiles, whose
  // single accumulator buffer exposes both passes, lose to the two kernels at 12 800 x 2048 -> 512).
  (void)M;
  (void)N;
  (void)K;
  (void)sms;
  return kPlanPair256S4E8;
}
static int rowquant_parts(int plan, int64_t N) {
  return (int)ceil_div(N, kGemmPlanBn[plan]) * (kGemmPlanEw[plan] / 4);
}
template <int BN, int STAGES, int EW>
static int launch_rowquant_cfg(const int8_t* a, const void* b, float* y, int64_t ldy, const GemmParams& p, cudaStream_t st) {
  if (p.small_acc) return launch_qgemm_inst<BN, STAGES, EW, false, false, kAccInt32Small, false, true, true>(a, b, y, ldy, p, st);
  return launch_qgemm_inst<BN, STAGES, EW, false, false, kAccInt32, false, true, true>(a, b, y, ldy, p, st);
}
static int launch_qgemm_rowquant(int plan, const int8_t* a, const void* b, float* y, int64_t ldy, GemmParams p, cudaStream_t st) {
  if (p.act != AQT_ACT_NONE && p.act != AQT_ACT_SWISH) return AQT_ERR_UNSUPPORTED;
  if (p.M <= kBM || p.kind != 0) return AQT_ERR_UNSUPPORTED;
  p.exchange_parts = rowquant_parts(plan, p.N);
  if (plan != kPlanPair256S4E8) return AQT_ERR_UNSUPPORTED;
  return launch_rowquant_cfg<256, 4, 8>(a, b, y, ldy, p, st);
}

static GemmShape gemm_shape_of(const GemmParams& p) {
  GemmShape g;
  g.M = p.M;
  g.N = p.N;
  g.K = p.K;
  g.act = p.act;
  g.kind = p.kind;
  g.batched = p.batch_tiles_m > 0;
  return g;
}

// forced_plan: kPlanNone lets the library choose.
static int launch_qgemm(const int8_t* a, const void* b, bool b_packed, float* y, int64_t ldy, const GemmParams& p, cudaStream_t st,
                        int forced_plan = kPlanNone) {
  const int sms = sm_count();
  if (sms <= 0) return AQT_ERR_CUDA;
  const GemmShape g = gemm_shape_of(p);
  int plan = forced_plan;
  if (plan != kPlanNone) {
    if (!gemm_plan_takes(plan, g, sms)) return AQT_ERR_UNSUPPORTED;
  } else {
    plan = plan_qgemm(g, sms);
  }
  return launch_qgemm_plan(plan, a, b, b_packed, y, ldy, p, st);
}

}  // namespace aqt
