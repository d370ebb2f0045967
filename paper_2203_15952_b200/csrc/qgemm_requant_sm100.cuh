// Integer GEMM whose epilogue quantizes its own output for the next layer (sm_100a).
//
//   acc = xq * wq^T (int32, TMEM);  u = residual + residual_scale * act(fma(float(acc) * s_x, s_w, bias))
//   amax[m] = max_n |u[m][n]|;  s_out[m] = amax[m] / qmax;  q_out[m][n] = round(u[m][n] / s_out[m])
//
// i.e. the dynamic quantizer of Fig. 2 of the paper applied to the layer's output rows before they
// ever leave the SM: the fp32 tensor between two quantized layers is neither written nor read
// back (it is written too only when the caller asks for it, e.g. for a residual stream).
//
// A row's abs-max spans all N output columns, i.e. several CTAs.  The grid is made of groups of
// tiles_n CTAs; the CTAs of a group own the n-tiles of the same m-tile at about the same time
// (weight stationary, K <= 512 or 1024: each keeps its weight slab resident) and exchange row maxima
// through global memory, one 64-bit word per (m-tile, n-tile, row): the maximum's bit pattern below a
// tag that identifies this execution, so a word is its own validity and nothing is cleared,
// counted or fenced.
//   epilogue warps    four sets of four warps (one warp per TMEM lane quadrant); set s owns
//                     accumulator buffer s and every fourth tile, all 128 columns of it:
//                       pass 1  accumulators -> u (registers) -> row maxima; u goes back into the
//                               TMEM columns it came from; the maxima are published
//                       wait    for the group's other CTAs (the exchange warps do the polling)
//                       pass 2  scale from the final maximum, u from TMEM, codes, stores; the TMEM
//                               buffer goes back to the MMA
//                     The four warps on a scheduler thus sit in four different phases of four
//                     different tiles, which is what keeps the special-function unit (pass 1 of a
//                     Swish tile) and the other pipes (pass 2) busy at the same time.
//   exchange warps    two, one per half of the rows: for each tile in turn read the words of all
//                     n-tiles (all requests in flight together), again until every one is valid,
//                     and leave the final maximum of each row in shared memory
// All CTAs of a group must be resident at once (they wait on one another): the grid never exceeds
// one CTA per SM.  Every wait is bounded as in the plain GEMM.
#pragma once

#include "qgemm_sm100.cuh"
#include "row_quant_epilogue.cuh"

namespace aqt {

struct RequantParams {
  GemmParams g;         // act: NONE or SWISH
  uint8_t* q_out;       // codes of the output: int8 [M, N] or packed nibbles [M, N/2], dense
  float* s_out;         // [M] scales of the output rows
  uint64_t* exchange;   // [tiles_m][tiles_n][128] words: (launch tag << 32) | bit pattern of a CTA's row maximum
  uint32_t* generation; // [groups] counters behind the words: each group of CTAs bumps its own when it has finished
  uint32_t tag;         // tag of this call (no other call of the process uses it); a word counts once its upper half
                        // equals this tag mixed with the group's generation, which differs on every execution of the call
  int qmax_out;         // 127 or 7
  int rounding;
  int pack_out;         // 1: two 4-bit codes per byte
};

// DEEP: the resident weight slab holds eight k-blocks (K <= 1024, the d = 1024 encoder's first
// FFN layers and pointwise 1) instead of four.  That leaves no room for the fp32 staging buffers
// or for the packed weights, so this form writes codes and scales only and reads int8 weights
// (4-bit ones are sign-extended into the workspace beforehand).
constexpr int kRequantDeepKBlocks = 8;
template <bool WITH_Y, bool DEEP = false>
struct RequantCfg {
  static_assert(!(DEEP && WITH_Y), "the deep-K form has no room for fp32 staging");
  static constexpr int kKBlocks = DEEP ? kRequantDeepKBlocks : kWsMaxKBlocks;
  static constexpr int BN = 128;
  static constexpr int EW = 16;
  static constexpr int kThreads = 32 * (2 + EW + 2);  // producer, MMA issuer, epilogue warps, two exchange warps
  static constexpr int kStages = (WITH_Y || DEEP) ? 5 : 7;
  static constexpr int kABytes = kBM * kBK;
  static constexpr int kBBytes = BN * kBK;
  static constexpr int kResidentBytes = kKBlocks * kBBytes;
  static constexpr int kYBytes = WITH_Y ? EW * kStageBufBytes : 0;
  static constexpr int kPackedBBytes = DEEP ? 0 : kWsMaxKBlocks * BN * 64;  // packed weights wait here for the unpack
  static constexpr int kEpiBytes = kYBytes > kPackedBBytes ? kYBytes : kPackedBBytes;
  static constexpr int kScaleBytes = 2 * BN * 4;
  static constexpr int kTmemCols = 4 * BN;
  static constexpr int kSmemBytes = kStages * kABytes + kResidentBytes + kEpiBytes + kScaleBytes + 1024;
  static_assert(kSmemBytes + 13312 <= 232448, "must fit the 227 KB a CTA can opt into");
};

// 32 lanes x 16 consecutive 32-bit columns (the GLU form: a warp owns 16 value and 16 gate columns).
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// dequant32 / swish32 of qgemm_sm100.cuh on 16 columns.
template <int ACCK>
__device__ __forceinline__ void dequant16(const uint32_t (&acc)[16], float sx, uint32_t sw_smem, uint32_t b_smem, float (&z)[16]) {
  const float2 sx2 = make_float2(sx, sx);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
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
__device__ __forceinline__ void swish16(float (&a)[16]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float2 z = make_float2(a[2 * j], a[2 * j + 1]);
    const float2 t = __fmul2_rn(z, make_float2(-1.4426950408889634f, -1.4426950408889634f));
    const float2 d = __fadd2_rn(make_float2(1.0f, 1.0f), make_float2(ex2_approx(t.x), ex2_approx(t.y)));
    const float2 y = __fmul2_rn(z, make_float2(rcp_approx(d.x), rcp_approx(d.y)));
    a[2 * j] = y.x;
    a[2 * j + 1] = y.y;
  }
}

// One slot of shared-memory exchange state (final row maxima, hand-over barriers) per accumulator
// buffer, i.e. per set of epilogue warps: tile i of a CTA uses buffer and slot i mod 4.
constexpr int kSlots = 4;
constexpr int kExchangeBatch = 16;  // n-tiles whose words an exchange warp asks for at once (one 16-byte load each per lane)

// Called between polls of a bounded wait: false once the CTA is aborting or the limit has passed
// (which then sets both the CTA's abort flag and the device status word).
__device__ __forceinline__ bool keep_waiting(volatile int* abort_flag, uint64_t t_start) {
  if (*abort_flag) return false;
  if (global_timer_ns() - t_start > kWaitLimitNs) {
    *abort_flag = 1;
    atomicExch(&g_device_status, AQT_ERR_TIMEOUT);
    return false;
  }
  return true;
}

// GLU: a tile's 128 weight rows are 64 value channels and their 64 gate channels; it yields 64
// output columns u = v * sigmoid(g) (then Swish for AQT_ACT_GLU_SWISH), 16 per epilogue warp.
// The GLU form writes codes and scales only (no fp32 output, no residual, no nibble packing).
template <bool BPACK, bool SMALL, bool WITH_Y, int ROUNDING, bool PACK_OUT, bool GLU = false, bool DEEP = false>
__global__ void __launch_bounds__(32 * 20, 1)
qgemm_requant_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_y,
                     const __grid_constant__ CUtensorMap tm_r, const RequantParams rp) {
  using Cfg = RequantCfg<WITH_Y, DEEP>;
  constexpr int BN = Cfg::BN, EW = Cfg::EW, STAGES = Cfg::kStages, HALF = BN / 2;
  static_assert(!(DEEP && BPACK), "the deep-K form reads int8 weights");
  static_assert(!GLU || (!WITH_Y && !PACK_OUT), "the GLU form writes int8 codes and scales only");
  const GemmParams& p = rp.g;
  const int n_out = GLU ? p.N / 2 : p.N;  // output columns

  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[STAGES];
  __shared__ uint64_t empty_bar[STAGES];
  __shared__ uint64_t tmem_full_bar[4];
  __shared__ uint64_t tmem_empty_bar[4];
  __shared__ uint64_t res_bar[EW];    // WITH_Y: residual tile landed in a warp's fp32 staging buffer
  __shared__ uint64_t b_loaded_bar;
  __shared__ uint64_t b_ready_bar;
  __shared__ __align__(16) uint32_t row_amax[kSlots][kBM];  // final row maxima (bit patterns) of a tile awaiting pass 2
  __shared__ uint64_t ctx_ready_bar[kSlots][2];  // an exchange warp has filled its half of row_amax[.]
  __shared__ uint64_t ctx_free_bar[kSlots][2];   // the set's two warps on that half of the rows have read theirs
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t smem_ring = smem_base;
  const uint32_t smem_res_b = smem_ring + STAGES * Cfg::kABytes;
  const uint32_t smem_epi = smem_res_b + Cfg::kResidentBytes;  // packed weights before the unpack, then (WITH_Y) fp32 staging
  const uint32_t smem_scale = smem_epi + Cfg::kEpiBytes;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint64_t t_start = global_timer_ns();

  // this CTA's n-tile and its group's m-tiles
  const int tn = blockIdx.x % p.tiles_n;
  const int group = blockIdx.x / p.tiles_n;
  const int groups = gridDim.x / p.tiles_n;
  const int n_my = group < p.tiles_m ? (p.tiles_m - group + groups - 1) / groups : 0;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b);
    if (WITH_Y) tma_prefetch_desc(&tm_y);
    if (WITH_Y && p.residual != nullptr) tma_prefetch_desc(&tm_r);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < 4; ++b) {
      mbar_init(smem_u32(&tmem_full_bar[b]), 1);
      mbar_init(smem_u32(&tmem_empty_bar[b]), 4);  // the four warps of the set that owns the buffer
    }
    for (int w = 0; w < EW; ++w) mbar_init(smem_u32(&res_bar[w]), 1);
    mbar_init(smem_u32(&b_loaded_bar), 1);
    mbar_init(smem_u32(&b_ready_bar), EW);
    for (int b = 0; b < kSlots; ++b) {
      for (int h = 0; h < 2; ++h) {
        mbar_init(smem_u32(&ctx_ready_bar[b][h]), 1);
        mbar_init(smem_u32(&ctx_free_bar[b][h]), 2);
      }
    }
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
    tmem_relinquish();
  }
  // Everything above touched only this CTA's own state; from here on global memory is read.  The
  // weights (codes, scales, bias) may be read before the kernel ahead of this one in the stream has
  // finished if the caller says they were complete before that kernel was enqueued (static_w): the
  // weight slab then loads and unpacks while that kernel drains, and every role waits for it only
  // before its first access to anything else.
  const bool early_w = p.static_w != 0;
  if (!early_w) grid_dependency_wait();
  for (int t = threadIdx.x; t < BN; t += blockDim.x) {
    // scales and biases of the tile's weight rows: (GLU) values first, then gates
    const int n = !GLU ? tn * BN + t : (t < HALF ? tn * HALF + t : p.N / 2 + tn * HALF + (t - HALF));
    const int limit = (GLU && t < HALF) ? p.N / 2 : p.N;
    float wv = 0.0f, bv = 0.0f;
    if (n < limit) {
      wv = __ldg(p.s_w + n);
      if (p.bias != nullptr) bv = __ldg(p.bias + n);
    }
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_scale + t * 4), "f"(wv) : "memory");
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_scale + (BN + t) * 4), "f"(bv) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      {
        const int row0 = GLU ? tn * HALF : tn * BN, row1 = GLU ? p.N / 2 + tn * HALF : tn * BN + HALF;
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
      if (early_w) grid_dependency_wait();  // the activation codes come from the kernel ahead
      for (int i = 0; ok && i < n_my; ++i) {
        const int tm = group + i * groups;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1, &abort_flag, t_start)) { ok = false; break; }
          const uint32_t bar = smem_u32(&full_bar[s]);
          mbar_arrive_expect_tx(bar, Cfg::kABytes);
          tma_load_2d(smem_ring + s * Cfg::kABytes, &tm_a, kb * kBK, tm * kBM, bar);
        }
      }
      grid_dependents_launch();  // every load of this CTA has been issued: the next kernel may be scheduled behind it
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_i8(BN, kBM);
      uint32_t it = 0;
      bool ok = mbar_wait(smem_u32(BPACK ? &b_ready_bar : &b_loaded_bar), 0, &abort_flag, t_start);
      for (int i = 0; ok && i < n_my; ++i) {
        const uint32_t buf = i & 3, aph = (i >> 2) & 1;
        if (!mbar_wait(smem_u32(&tmem_empty_bar[buf]), aph ^ 1, &abort_flag, t_start)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!mbar_wait(smem_u32(&full_bar[s]), ph, &abort_flag, t_start)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = smem_desc_k_major_sw128(smem_ring + s * Cfg::kABytes);
          const uint64_t b_desc = smem_desc_k_major_sw128(smem_res_b + kb * Cfg::kBBytes);
#pragma unroll
          for (int kk = 0; kk < kBK / kMmaK; ++kk) tc_mma_i8(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          tc_commit(smem_u32(&empty_bar[s]));
        }
        if (ok) tc_commit(smem_u32(&tmem_full_bar[buf]));
      }
    }
  } else if (warp >= 2 + EW) {
    // ------------------------------------------------------------------ exchange warps
    // Two warps, each for one half of the tile's rows: lane l of warp h owns rows 64h + 2l and
    // 64h + 2l + 1, i.e. one 16-byte load (two words) per n-tile, kExchangeBatch of them in flight.
    const int xh = warp - (2 + EW);
    bool ok = true;
    if (early_w) grid_dependency_wait();
    // Tag of this execution's exchange words.  A replayed CUDA graph repeats the call's own tag, so the
    // group's generation counter goes into it: every CTA of the group reads it at its start, and the
    // group's first CTA bumps it after its last tile, which it cannot finish before all of them have started.
    const uint32_t tag = mix_tag(rp.tag, __ldcg(rp.generation + group));
    for (int i = 0; ok && i < n_my; ++i) {
      const int tm = group + i * groups;
      const uint32_t par = i % kSlots, ph = (i / kSlots) & 1;
      if (!mbar_wait(smem_u32(&ctx_free_bar[par][xh]), ph ^ 1, &abort_flag, t_start)) break;
      const uint64_t* xt = rp.exchange + (size_t)tm * p.tiles_n * kBM + 64 * xh + 2 * lane;
      uint2 m2 = make_uint2(0u, 0u);
      for (int t0 = 0; ok && t0 < p.tiles_n; t0 += kExchangeBatch) {
        // all loads of the batch in flight at once; the whole batch is asked for again until every word carries this launch's tag
        for (uint32_t spin = 1;; ++spin) {
          ulonglong2 w[kExchangeBatch];
#pragma unroll
          for (int t = 0; t < kExchangeBatch; ++t) {
            const uint64_t none = (uint64_t)tag << 32;  // a maximum of zero
            w[t] = t0 + t < p.tiles_n ? ld_relaxed_gpu_2x64(xt + (size_t)(t0 + t) * kBM) : make_ulonglong2(none, none);
          }
          bool all = true;
          uint2 b2 = make_uint2(0u, 0u);
#pragma unroll
          for (int t = 0; t < kExchangeBatch; ++t) {
            all = all && (uint32_t)(w[t].x >> 32) == tag && (uint32_t)(w[t].y >> 32) == tag;
            b2.x = max(b2.x, (uint32_t)w[t].x);
            b2.y = max(b2.y, (uint32_t)w[t].y);
          }
          if (__all_sync(0xffffffffu, all)) {
            m2.x = max(m2.x, b2.x);
            m2.y = max(m2.y, b2.y);
            break;
          }
          if ((spin & 0xF) == 0 && !__all_sync(0xffffffffu, keep_waiting(&abort_flag, t_start))) { ok = false; break; }  // warp-uniform
        }
      }
      if (!__all_sync(0xffffffffu, ok)) break;
      // final maxima of this warp's rows for the epilogue warps
      *reinterpret_cast<uint2*>(&row_amax[par][64 * xh + 2 * lane]) = m2;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctx_ready_bar[par][xh]));
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    // Four sets of four warps, one warp of a set per TMEM lane quadrant (hence one per scheduler).
    // Set s owns accumulator buffer s and with it every fourth tile of this CTA, all of its
    // columns: pass 1 chunk by chunk, publication of the rows' maxima straight from registers
    // (a thread has seen its whole row of the tile, so nothing is merged across warps), the wait
    // for the other n-tiles' maxima, pass 2.  The four warps that share a scheduler therefore work
    // on four different tiles in four different phases: while one is on the special-function unit
    // (pass 1 of a Swish tile is bound by it), the others issue multiply-adds and byte permutes
    // (pass 2), wait for the exchange, or wait for the tensor core.
    const int ew = warp - 2;
    const int quad = warp & 3;  // TMEM lane quadrant this warp may access
    const int set = ew >> 2;    // accumulator buffer and tile residue (mod 4) of this warp
    constexpr int CW = GLU ? 16 : 32;  // output columns per chunk; four chunks per tile
    const int row_in_tile = quad * 32 + lane;
    const uint32_t y_buf = smem_epi + ew * kStageBufBytes;
    const bool has_res = WITH_Y && p.residual != nullptr;
    const int oc0 = tn * (GLU ? HALF : BN);  // first output column of this CTA's tiles
    bool ok = true;

    if (BPACK) {
      // sign-extend the packed weights into the resident slab (layout of a swizzled int8 load)
      ok = mbar_wait(smem_u32(&b_loaded_bar), 0, &abort_flag, t_start);
      if (ok) {
        const int pieces = p.k_blocks * BN * 4;
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
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&b_ready_bar));
        ok = mbar_wait(smem_u32(&b_ready_bar), 0, &abort_flag, t_start);  // staging area free for the fp32 output
      }
    }

    if (early_w) grid_dependency_wait();  // scales of the activations, residual, outputs: everything but the weights
    const uint32_t tag = mix_tag(rp.tag, __ldcg(rp.generation + group));  // see the exchange warps
    uint32_t res_count = 0;  // residual boxes this warp has consumed (phase of its barrier)
    if (ok && has_res && lane == 0 && set < n_my) {
      const int r0 = (group + set * groups) * kBM + quad * 32;
      mbar_arrive_expect_tx(smem_u32(&res_bar[ew]), kStageBufBytes);
      tma_load_2d(y_buf, &tm_r, oc0 < n_out ? oc0 : 0, r0 < p.M ? r0 : 0, smem_u32(&res_bar[ew]));
    }

    const uint32_t buf = (uint32_t)set;
    const uint32_t tbase = tmem_base + buf * BN + ((uint32_t)(quad * 32) << 16);
    for (int i = set; ok && i < n_my; i += 4) {
      const int tm = group + i * groups;
      const uint32_t aph = (uint32_t)(i >> 2) & 1u;
      const int row0_warp = tm * kBM + quad * 32;
      const int m = row0_warp + lane;
      const float sx = (p.s_x_kind == AQT_SCALE_ROW) ? (m < p.M ? __ldg(p.s_x + m) : 0.0f) : __ldg(p.s_x);
      if (!mbar_wait(smem_u32(&tmem_full_bar[buf]), aph, &abort_flag, t_start)) { ok = false; break; }
      tc_fence_after();

      // -------------------------------------------------------------- pass 1: u, row maxima; u back to TMEM
      float amax = 0.0f;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        const int col = c * CW;
        const bool cols_ok = oc0 + col < n_out;  // columns beyond N contribute nothing
        const uint32_t c_sw = smem_scale + (uint32_t)col * 4, c_bias = c_sw + BN * 4;
        if constexpr (GLU) {
          // gates first: g = sigmoid(z_gate); then the values are scaled by it
          uint32_t accv[16], accg[16];
          float av[16], g[16];
          tmem_ld_32x16(tbase + HALF + col, accg);
          tmem_ld_32x16(tbase + col, accv);
          tmem_ld_wait();
          dequant16<SMALL>(accg, sx, c_sw + HALF * 4, c_bias + HALF * 4, g);
#pragma unroll
          for (int j = 0; j < 16; ++j) g[j] = sigmoid_f(g[j]);
          dequant16<SMALL>(accv, sx, c_sw, c_bias, av);
#pragma unroll
          for (int j = 0; j < 16; ++j) av[j] = av[j] * g[j];
          if (p.act == AQT_ACT_GLU_SWISH) swish16(av);
          float cmax = 0.0f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            cmax = fmaxf(cmax, fabsf(av[j]));
            accv[j] = __float_as_uint(av[j]);
          }
          if (cols_ok) amax = fmaxf(amax, cmax);
          tmem_st_32x16(tbase + col, accv);  // u replaces the value accumulators
        } else {
          uint32_t acc[32];
          float a[32];
          tmem_ld_32x32(tbase + col, acc);
          tmem_ld_wait();
          dequant32<SMALL>(acc, sx, c_sw, c_bias, a);
          if (p.act == AQT_ACT_SWISH) swish32(a);
          if (has_res) {
            if (!mbar_wait(smem_u32(&res_bar[ew]), res_count & 1u, &abort_flag, t_start)) { ok = false; break; }
            ++res_count;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint32_t src = y_buf + lane * 128 + ((j ^ (lane & 7)) << 4);
              float r0, r1, r2, r3;
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r0), "=f"(r1), "=f"(r2), "=f"(r3) : "r"(src) : "memory");
              a[4 * j + 0] = __fmaf_rn(p.residual_scale, a[4 * j + 0], r0);
              a[4 * j + 1] = __fmaf_rn(p.residual_scale, a[4 * j + 1], r1);
              a[4 * j + 2] = __fmaf_rn(p.residual_scale, a[4 * j + 2], r2);
              a[4 * j + 3] = __fmaf_rn(p.residual_scale, a[4 * j + 3], r3);
            }
            __syncwarp();  // every lane has read its residual row before the buffer is overwritten
          }
          float cmax = 0.0f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            cmax = fmaxf(cmax, fabsf(a[j]));
            acc[j] = __float_as_uint(a[j]);
          }
          if (cols_ok) amax = fmaxf(amax, cmax);
          tmem_st_32x32(tbase + col, acc);  // u replaces the accumulators it was made from
          if (WITH_Y) {
            if (!has_res) {
              if (lane == 0) tma_store_wait_read<0>();  // the previous chunk's bulk store has read the buffer out
              __syncwarp();
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint32_t dst = y_buf + lane * 128 + ((j ^ (lane & 7)) << 4);
              asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(a[4 * j]), "f"(a[4 * j + 1]), "f"(a[4 * j + 2]),
                           "f"(a[4 * j + 3])
                           : "memory");
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (cols_ok && row0_warp < p.M) tma_store_2d(&tm_y, y_buf, oc0 + col, row0_warp);
              tma_store_commit();
              if (has_res) {
                // the next chunk's residual goes into the same buffer once this store has read it out
                tma_store_wait_read<0>();
                const bool more_here = c + 1 < 4;
                if (more_here || i + 4 < n_my) {
                  const int ncol = oc0 + (more_here ? col + CW : 0);
                  const int nr = (more_here ? tm : tm + 4 * groups) * kBM + quad * 32;
                  mbar_arrive_expect_tx(smem_u32(&res_bar[ew]), kStageBufBytes);
                  tma_load_2d(y_buf, &tm_r, ncol < n_out ? ncol : 0, nr < p.M ? nr : 0, smem_u32(&res_bar[ew]));
                }
              }
            }
          }
        }
      }
      if (!ok) break;
      // this CTA's maxima of the tile's rows, each tagged valid: one word per row, straight from the registers
      st_relaxed_gpu_64(rp.exchange + ((size_t)tm * p.tiles_n + tn) * kBM + row_in_tile, ((uint64_t)tag << 32) | __float_as_uint(amax));

      // -------------------------------------------------------------- pass 2: scale, codes
      if (!mbar_wait(smem_u32(&ctx_ready_bar[set][quad >> 1]), aph, &abort_flag, t_start)) { ok = false; break; }
      const float amax_row = __uint_as_float(row_amax[set][row_in_tile]);
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctx_free_bar[set][quad >> 1]));
      const ScaleCtx sc = make_scale_ctx(amax_row, rp.qmax_out);
      if (tn == 0 && m < p.M) rp.s_out[m] = sc.s;
      tmem_st_wait();  // this warp's stores of pass 1
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        const int col = c * CW;
        const int oc = oc0 + col;
        const bool cols_ok = oc < n_out;
        if constexpr (GLU) {
          uint32_t u[16], w[4];
          tmem_ld_32x16(tbase + col, u);
          tmem_ld_wait();
          if (c == 3) {
            // the tile has been read out by this warp: the accumulator buffer goes back to the MMA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tmem_empty_bar[buf]));
          }
          codes_of<ROUNDING, false, 16>(u, sc, rp.qmax_out, w);
          // 16 consecutive codes of the row: one 16-byte store
          if (m < p.M && cols_ok) *reinterpret_cast<uint4*>(rp.q_out + (size_t)m * n_out + oc) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
          uint32_t u[32], w[8];
          tmem_ld_32x32(tbase + col, u);
          tmem_ld_wait();
          if (c == 3) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tmem_empty_bar[buf]));
          }
          codes_of<ROUNDING, PACK_OUT, 32>(u, sc, rp.qmax_out, w);
          // Each thread holds 32 consecutive codes of its row: one or two 16-byte stores, each a
          // whole 32-byte sector (or half of one for packed nibbles), straight to global memory.
          if (m < p.M && cols_ok) {
            if (PACK_OUT) {
              uint4* dst = reinterpret_cast<uint4*>(rp.q_out + (size_t)m * (p.N / 2) + oc / 2);
              *dst = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
              uint4* dst = reinterpret_cast<uint4*>(rp.q_out + (size_t)m * p.N + oc);
              dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
              if (oc + 16 < p.N) dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
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
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) {
    }
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
  if (tn == 0 && threadIdx.x == 0) rp.generation[group] = __ldcg(rp.generation + group) + 1u;
}

// Bytes of the exchange area: one 64-bit word per m-tile, n-tile and row for this kernel, or per
// row (padded to the 256 rows of a pair tile) and column part for the CTA-pair kernel with the
// row-quantizing epilogue (at most one part per 64 columns, at least two), then the generation counters.
static size_t requant_exchange_bytes(int64_t M, int64_t N) {
  const size_t tiles_m = (size_t)ceil_div(M, kBM);
  const size_t ws_form = tiles_m * (size_t)ceil_div(N, 128) * kBM * 8;
  const size_t parts = (size_t)ceil_div(N, 64) < 2 ? 2 : (size_t)ceil_div(N, 64);
  const size_t pair_form = (size_t)ceil_div(M, 2 * kBM) * 2 * kBM * parts * 8;
  return round_up((ws_form > pair_form ? ws_form : pair_form) + (size_t)kMaxGroups * 4, 256);
}

// True if this kernel takes the call: K <= 512; NONE / Swish in every form, the GLU forms when
// only int8 codes and scales are asked for (no fp32 output, hence no residual, no nibble packing).
static bool requant_applies(int64_t M, int64_t N, int64_t K, int act, bool with_y, bool pack_out) {
  const int sms = sm_count() > 0 ? sm_count() : kDefaultSms;
  if (!(M > 0 && ceil_div(N, 128) <= sms)) return false;
  const bool glu = !(act == AQT_ACT_NONE || act == AQT_ACT_SWISH);
  if (ceil_div(K, kBK) <= kWsMaxKBlocks) return !glu || (!with_y && !pack_out);
  // 512 < K <= 1024: codes and scales only
  return ceil_div(K, kBK) <= kRequantDeepKBlocks && !with_y && (!glu || !pack_out);
}

template <bool BPACK, bool SMALL, bool WITH_Y, int ROUNDING, bool PACK_OUT, bool GLU = false, bool DEEP = false>
static int launch_requant_inst(const int8_t* a, const void* b, void* q_out, float* y, int64_t ldy, RequantParams rp,
                               void* exchange, cudaStream_t st) {
  using Cfg = RequantCfg<WITH_Y, DEEP>;
  GemmParams& p = rp.g;
  p.tiles_m = (int)ceil_div(p.M, kBM);
  p.tiles_n = (int)ceil_div(p.N, Cfg::BN);
  p.k_blocks = (int)ceil_div(p.K, kBK);
  const int sms = sm_count();
  if (sms <= 0) return AQT_ERR_CUDA;
  if (p.k_blocks > Cfg::kKBlocks || p.tiles_n > sms) return AQT_ERR_UNSUPPORTED;
  rp.exchange = reinterpret_cast<uint64_t*>(exchange);
  rp.generation = reinterpret_cast<uint32_t*>(rp.exchange + (size_t)p.tiles_m * p.tiles_n * kBM);
  rp.tag = next_launch_tag();

  CUtensorMap tm_a, tm_b, tm_y, tm_r;
  int rc = make_map_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, a, (uint64_t)p.M, (uint64_t)p.K, (uint64_t)p.K, kBM, kBK);
  if (rc != AQT_OK) return rc;
  if (BPACK) rc = make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b, (uint64_t)p.N, (uint64_t)p.K / 2, (uint64_t)p.K / 2, Cfg::BN / 2, 64, 0);
  else rc = make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b, (uint64_t)p.N, (uint64_t)p.K, (uint64_t)p.K, Cfg::BN / 2, kBK);
  if (rc != AQT_OK) return rc;
  rp.q_out = reinterpret_cast<uint8_t*>(q_out);
  tm_y = tm_a;
  tm_r = tm_a;
  if (WITH_Y) {
    rc = make_map_2d(&tm_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, y, (uint64_t)p.M, (uint64_t)p.N, (uint64_t)ldy * 4, kStoreBoxRows, kStoreBoxCols);
    if (rc != AQT_OK) return rc;
    if (p.residual != nullptr) {
      rc = make_map_2d(&tm_r, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, p.residual, (uint64_t)p.M, (uint64_t)p.N, (uint64_t)p.ldr * 4, kStoreBoxRows,
                       kStoreBoxCols);
      if (rc != AQT_OK) return rc;
    }
  }
  auto kernel = qgemm_requant_kernel<BPACK, SMALL, WITH_Y, ROUNDING, PACK_OUT, GLU, DEEP>;
  static std::atomic<uint64_t> smem_opted_in{0};
  rc = ensure_dynamic_smem(kernel, Cfg::kSmemBytes, smem_opted_in);
  if (rc != AQT_OK) return rc;
  int groups = sms / p.tiles_n;
  if (groups > p.tiles_m) groups = p.tiles_m;
  // The CTAs of a group wait on one another, so all of them must get an SM: the grid never exceeds
  // one CTA per SM (each takes most of an SM's shared memory), and CTAs of the kernel before it in
  // the stream never wait on anything, so the SMs they hold become free.  Should another stream keep
  // SMs occupied for seconds, the bounded waits give up and report AQT_ERR_TIMEOUT.
  return launch_pdl(kernel, dim3((unsigned)(groups * p.tiles_n), 1, 1), dim3(Cfg::kThreads, 1, 1), Cfg::kSmemBytes, st, 1, tm_a, tm_b,
                    tm_y, tm_r, rp);
}

// a: int8 [M, K]; b: int8 [N, K] or (b_packed) nibbles [N, K/2]; y may be null (then no fp32 output
// and no residual).  exchange: requant_exchange_bytes(M, N) bytes.
static int launch_requant(const int8_t* a, const void* b, bool b_packed, void* q_out, float* y, int64_t ldy, const RequantParams& rp,
                          void* exchange, cudaStream_t st) {
  const bool small = rp.g.small_acc != 0;
  const bool glu = rp.g.act == AQT_ACT_GLU || rp.g.act == AQT_ACT_GLU_SWISH;
  if (ceil_div(rp.g.K, kBK) > kWsMaxKBlocks) {
    // deep-K form: int8 weights, codes and scales only
    if (y != nullptr || b_packed || (glu && rp.pack_out)) return AQT_ERR_UNSUPPORTED;
#define AQT_RQ_DEEP(SM, PK, GL)                                                                                                   \
  (rp.rounding == AQT_ROUND_HALF_UP_FLOOR ? launch_requant_inst<false, SM, false, AQT_ROUND_HALF_UP_FLOOR, PK, GL, true>(a, b, q_out, y, ldy, rp, exchange, st) \
                                          : launch_requant_inst<false, SM, false, AQT_ROUND_NEAREST_EVEN, PK, GL, true>(a, b, q_out, y, ldy, rp, exchange, st))
    if (glu) return small ? AQT_RQ_DEEP(true, false, true) : AQT_RQ_DEEP(false, false, true);
    if (rp.pack_out) return small ? AQT_RQ_DEEP(true, true, false) : AQT_RQ_DEEP(false, true, false);
    return small ? AQT_RQ_DEEP(true, false, false) : AQT_RQ_DEEP(false, false, false);
#undef AQT_RQ_DEEP
  }
  if (glu) {
    if (y != nullptr || rp.pack_out) return AQT_ERR_UNSUPPORTED;
#define AQT_RQ_GLU(BP, SM)                                                                                                        \
  (rp.rounding == AQT_ROUND_HALF_UP_FLOOR ? launch_requant_inst<BP, SM, false, AQT_ROUND_HALF_UP_FLOOR, false, true>(a, b, q_out, y, ldy, rp, exchange, st) \
                                          : launch_requant_inst<BP, SM, false, AQT_ROUND_NEAREST_EVEN, false, true>(a, b, q_out, y, ldy, rp, exchange, st))
    if (b_packed) return small ? AQT_RQ_GLU(true, true) : AQT_RQ_GLU(true, false);
    return small ? AQT_RQ_GLU(false, true) : AQT_RQ_GLU(false, false);
#undef AQT_RQ_GLU
  }
#define AQT_RQ(BP, SM, WY)                                                                                                 \
  (rp.pack_out ? (rp.rounding == AQT_ROUND_HALF_UP_FLOOR                                                                     \
                      ? launch_requant_inst<BP, SM, WY, AQT_ROUND_HALF_UP_FLOOR, true>(a, b, q_out, y, ldy, rp, exchange, st) \
                      : launch_requant_inst<BP, SM, WY, AQT_ROUND_NEAREST_EVEN, true>(a, b, q_out, y, ldy, rp, exchange, st)) \
               : (rp.rounding == AQT_ROUND_HALF_UP_FLOOR                                                                     \
                      ? launch_requant_inst<BP, SM, WY, AQT_ROUND_HALF_UP_FLOOR, false>(a, b, q_out, y, ldy, rp, exchange, st) \
                      : launch_requant_inst<BP, SM, WY, AQT_ROUND_NEAREST_EVEN, false>(a, b, q_out, y, ldy, rp, exchange, st)))
  if (y != nullptr) {
    if (b_packed) return small ? AQT_RQ(true, true, true) : AQT_RQ(true, false, true);
    return small ? AQT_RQ(false, true, true) : AQT_RQ(false, false, true);
  }
  if (b_packed) return small ? AQT_RQ(true, true, false) : AQT_RQ(true, false, false);
  return small ? AQT_RQ(false, true, false) : AQT_RQ(false, false, false);
#undef AQT_RQ
}

}  // namespace aqt
