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
// tiles_n CTAs; the CTAs of a group own the n-tiles of the same m-tile at the same time (weight
// stationary, K <= 512: each keeps its weight slab resident) and exchange row maxima through
// global memory, one word per (m-tile, n-tile, row):
//   pass 1 (tile j)   TMEM accumulators -> u (registers) -> row maxima; u goes back into the TMEM
//                     columns it came from; the last of the four warps that share a row quadrant
//                     merges their maxima and stores them, tagged valid in the sign bit (a
//                     maximum is never negative), into the CTA's words of the exchange area
//   pass 2 (tile j-1) reads the row's words of all n-tiles (requested before pass 1 of tile j, so
//                     the round trip overlaps it), waits for any that is not yet valid, forms the
//                     scale from the final maximum, u from TMEM, codes, TMA store; the TMEM
//                     buffer goes back to the MMA
// Every word carries its own validity, so no counter, fence or atomic on global memory is needed.
// Pass 2 of a tile runs after pass 1 of the next one, so the exchange has a tile's worth of time
// to complete; four TMEM buffers of 128 columns keep the tensor core two tiles ahead.
// All CTAs must be resident at once (they wait on one another): the launch is cooperative and
// the grid never exceeds one CTA per SM.  Every wait is bounded as in the plain GEMM.
#pragma once

#include "qgemm_sm100.cuh"

namespace aqt {

struct RequantParams {
  GemmParams g;         // act: NONE or SWISH
  float* s_out;         // [M] scales of the output rows
  uint32_t* exchange;   // [tiles_m][tiles_n][128]: bit pattern of a CTA's row maximum | 0x80000000; zero on entry
  int qmax_out;         // 127 or 7
  int rounding;
  int pack_out;         // 1: two 4-bit codes per byte
};

template <bool WITH_Y>
struct RequantCfg {
  static constexpr int BN = 128;
  static constexpr int EW = 16;
  static constexpr int kThreads = 32 * (2 + EW);
  static constexpr int kStages = WITH_Y ? 4 : 6;
  static constexpr int kABytes = kBM * kBK;
  static constexpr int kBBytes = BN * kBK;
  static constexpr int kResidentBytes = kWsMaxKBlocks * kBBytes;
  static constexpr int kCodeBufBytes = 32 * 32;                  // per warp: 32 rows x 32 codes
  static constexpr int kCodeBytes = EW * kCodeBufBytes;
  static constexpr int kYBytes = WITH_Y ? EW * kStageBufBytes : 0;
  static constexpr int kPackedBBytes = kWsMaxKBlocks * BN * 64;  // packed weights wait here for the unpack
  static constexpr int kEpiBytes = (kCodeBytes + kYBytes) > kPackedBBytes ? (kCodeBytes + kYBytes) : kPackedBBytes;
  static constexpr int kScaleBytes = 2 * BN * 4;
  static constexpr int kTmemCols = 4 * BN;
  static constexpr int kSmemBytes = kStages * kABytes + kResidentBytes + kEpiBytes + kScaleBytes + 1024;
  static_assert(kSmemBytes + 1024 <= 232448, "must fit the 227 KB a CTA can opt into");
};

__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
      "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
      "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t ld_relaxed_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_gpu(uint32_t* p, uint32_t v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

constexpr uint32_t kValidBit = 0x80000000u;
constexpr int kPrefetchWords = 16;  // exchange words per row requested ahead of pass 1 (covers N <= 2048)

// Bounded wait for an exchange word to become valid; `w` is what an earlier load returned.
__device__ __forceinline__ bool wait_valid(const uint32_t* p, uint32_t& w, volatile int* abort_flag, uint64_t t_start) {
  for (uint32_t spin = 1; (w & kValidBit) == 0u; ++spin) {
    w = ld_relaxed_gpu(p);
    if ((spin & 0x3F) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t_start > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(&g_device_status, AQT_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Codes of four values whose row scale constants are known (fast path of the quantizer: the
// correctly rounded quotient by one multiply and two fused multiply-adds).  Rounding by adding
// 1.5 * 2^23: the sum's low mantissa bits are the integer in two's complement, so the code's
// byte is the low byte of the sum's bit pattern.  Nearest-even is the add's own rounding; the
// figure's floor(v + 0.5) is the binary32 add of 0.5 followed by an add rounded towards minus
// infinity.  Exact for |v| < 2^22; here |v| <= 127 (1 + 2^-23).
template <int ROUNDING>
__device__ __forceinline__ uint32_t code_bits(float x, float s, float r) {
  const float q0 = __fmul_rn(x, r);
  const float e = __fmaf_rn(-q0, s, x);
  const float v = __fmaf_rn(e, r, q0);
  if (ROUNDING == AQT_ROUND_HALF_UP_FLOOR) return __float_as_uint(__fadd_rd(__fadd_rn(v, 0.5f), 12582912.0f));
  return __float_as_uint(__fadd_rn(v, 12582912.0f));
}
__device__ __forceinline__ uint32_t low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  const uint32_t lo = __byte_perm(a, b, 0x0040);
  const uint32_t hi = __byte_perm(c, d, 0x0040);
  return __byte_perm(lo, hi, 0x5410);
}
// Eight codes as nibbles (element 0 in the low nibble of byte 0) from two words of four bytes.
__device__ __forceinline__ uint32_t nibbles_of(uint32_t w0, uint32_t w1) {
  const uint32_t x0 = w0 & 0x0F0F0F0Fu, x1 = w1 & 0x0F0F0F0Fu;
  const uint32_t y0 = x0 | (x0 >> 4), y1 = x1 | (x1 >> 4);  // bytes 0 and 2 hold a pair each
  return __byte_perm(y0, y1, 0x6420);
}

// 32 values of one row -> 8 words of int8 codes (PACK: 4 words of nibbles).
template <int ROUNDING, bool PACK>
__device__ __forceinline__ void codes32(const uint32_t (&u)[32], const ScaleCtx& c, int qmax, uint32_t (&w)[8]) {
  if (c.fast) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      w[j] = low_bytes(code_bits<ROUNDING>(__uint_as_float(u[4 * j]), c.s, c.r), code_bits<ROUNDING>(__uint_as_float(u[4 * j + 1]), c.s, c.r),
                       code_bits<ROUNDING>(__uint_as_float(u[4 * j + 2]), c.s, c.r), code_bits<ROUNDING>(__uint_as_float(u[4 * j + 3]), c.s, c.r));
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      w[j] = low_bytes((uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j]), c, qmax),
                       (uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j + 1]), c, qmax),
                       (uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j + 2]), c, qmax),
                       (uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j + 3]), c, qmax));
  }
  if (PACK) {
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = nibbles_of(w[2 * j], w[2 * j + 1]);
  }
}

template <bool BPACK, bool SMALL, bool WITH_Y>
__global__ void __launch_bounds__(32 * 18, 1)
qgemm_requant_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_y,
                     const __grid_constant__ CUtensorMap tm_r, const RequantParams rp) {
  using Cfg = RequantCfg<WITH_Y>;
  constexpr int BN = Cfg::BN, EW = Cfg::EW, STAGES = Cfg::kStages, HALF = BN / 2;
  const GemmParams& p = rp.g;

  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[STAGES];
  __shared__ uint64_t empty_bar[STAGES];
  __shared__ uint64_t tmem_full_bar[4];
  __shared__ uint64_t tmem_empty_bar[4];
  __shared__ uint64_t res_bar[EW];    // WITH_Y: residual tile landed in a warp's fp32 staging buffer
  __shared__ uint64_t b_loaded_bar;
  __shared__ uint64_t b_ready_bar;
  __shared__ uint32_t amax_part[2][4][kBM];  // row maxima per column part of the tile in pass 1 (even / odd tiles)
  // Warps of a row quadrant that have written their part (running counts, even / odd tiles).  A warp
  // can be in pass 1 of tile j + 1 while another is still in pass 1 of tile j, but not of tile
  // j + 2 (its pass 2 of tile j needs this quadrant's maxima of tile j published): two counters.
  __shared__ uint32_t quad_arrivals[2][4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t smem_ring = smem_base;
  const uint32_t smem_res_b = smem_ring + STAGES * Cfg::kABytes;
  const uint32_t smem_epi = smem_res_b + Cfg::kResidentBytes;  // code staging, then (WITH_Y) fp32 staging
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
    tma_prefetch_desc(&tm_q);
    if (WITH_Y) tma_prefetch_desc(&tm_y);
    if (WITH_Y && p.residual != nullptr) tma_prefetch_desc(&tm_r);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < 4; ++b) {
      mbar_init(smem_u32(&tmem_full_bar[b]), 1);
      mbar_init(smem_u32(&tmem_empty_bar[b]), EW);
    }
    for (int w = 0; w < EW; ++w) mbar_init(smem_u32(&res_bar[w]), 1);
    mbar_init(smem_u32(&b_loaded_bar), 1);
    mbar_init(smem_u32(&b_ready_bar), EW);
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
    tmem_relinquish();
  }
  for (int t = threadIdx.x; t < BN; t += blockDim.x) {
    const int n = tn * BN + t;
    float wv = 0.0f, bv = 0.0f;
    if (n < p.N) {
      wv = __ldg(p.s_w + n);
      if (p.bias != nullptr) bv = __ldg(p.bias + n);
    }
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_scale + t * 4), "f"(wv) : "memory");
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_scale + (BN + t) * 4), "f"(bv) : "memory");
  }
  if (threadIdx.x < 8) quad_arrivals[threadIdx.x >> 2][threadIdx.x & 3] = 0u;
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
        const int row0 = tn * BN, row1 = tn * BN + HALF;
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
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int ew = warp - 2;
    const int quad = warp & 3;   // TMEM lane quadrant this warp may access
    const int cpart = ew >> 2;   // which 32 columns of the tile
    const int col = cpart * 32;
    const int row_in_tile = quad * 32 + lane;
    const uint32_t code_buf = smem_epi + ew * Cfg::kCodeBufBytes;
    const uint32_t y_buf = smem_epi + Cfg::kCodeBytes + ew * kStageBufBytes;
    const uint32_t c_sw = smem_scale + (uint32_t)col * 4, c_bias = c_sw + BN * 4;
    const bool has_res = WITH_Y && p.residual != nullptr;
    const int oc = tn * BN + col;  // first output column of this warp
    const bool cols_ok = oc < p.N;
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
        ok = mbar_wait(smem_u32(&b_ready_bar), 0, &abort_flag, t_start);  // staging area free for codes
      }
    }

    if (ok && has_res && lane == 0 && n_my > 0) {
      const int r0 = group * kBM + quad * 32;
      mbar_arrive_expect_tx(smem_u32(&res_bar[ew]), kStageBufBytes);
      tma_load_2d(y_buf, &tm_r, cols_ok ? oc : 0, r0 < p.M ? r0 : 0, smem_u32(&res_bar[ew]));
    }

    for (int i = 0; ok && i <= n_my; ++i) {
      // exchange words of tile i - 1 for this thread's row, one per n-tile: requested now, used in pass 2
      uint32_t xw[kPrefetchWords];
      const uint32_t* xrow = rp.exchange + (size_t)(group + (i > 0 ? i - 1 : 0) * groups) * p.tiles_n * kBM + row_in_tile;
      if (i >= 1) {
#pragma unroll
        for (int t = 0; t < kPrefetchWords; ++t) xw[t] = t < p.tiles_n ? ld_relaxed_gpu(xrow + (size_t)t * kBM) : kValidBit;
      }
      if (i < n_my) {
        // -------------------------------------------------------------- pass 1 of tile i
        const int tm = group + i * groups;
        const uint32_t buf = i & 3, aph = (i >> 2) & 1;
        const int row0_warp = tm * kBM + quad * 32;
        const int m = row0_warp + lane;
        const float sx = (p.s_x_kind == AQT_SCALE_ROW) ? (m < p.M ? __ldg(p.s_x + m) : 0.0f) : __ldg(p.s_x);
        if (!mbar_wait(smem_u32(&tmem_full_bar[buf]), aph, &abort_flag, t_start)) { ok = false; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + buf * BN + ((uint32_t)(quad * 32) << 16) + col;
        uint32_t acc[32];
        float a[32];
        tmem_ld_32x32(taddr, acc);
        tmem_ld_wait();
        dequant32<SMALL>(acc, sx, c_sw, c_bias, a);
        if (p.act == AQT_ACT_SWISH) {
#pragma unroll
          for (int j = 0; j < 32; ++j) a[j] = a[j] * sigmoid_f(a[j]);
        }
        if (has_res) {
          if (!mbar_wait(smem_u32(&res_bar[ew]), i & 1, &abort_flag, t_start)) { ok = false; break; }
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
          __syncwarp();
        }
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          amax = fmaxf(amax, fabsf(a[j]));
          acc[j] = __float_as_uint(a[j]);
        }
        tmem_st_32x32(taddr, acc);
        // this warp's part of the row maxima (columns beyond N contribute nothing)
        amax_part[i & 1][cpart][row_in_tile] = cols_ok ? __float_as_uint(amax) : 0u;
        tmem_st_wait();
        __syncwarp();
        int last = 0;
        if (lane == 0) {
          __threadfence_block();
          last = (atomicAdd(&quad_arrivals[i & 1][quad], 1u) & 3u) == 3u ? 1 : 0;
          __threadfence_block();
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          // the last of the quadrant's four warps publishes the CTA's maxima of these 32 rows
          const uint32_t v = max(max(amax_part[i & 1][0][row_in_tile], amax_part[i & 1][1][row_in_tile]),
                                 max(amax_part[i & 1][2][row_in_tile], amax_part[i & 1][3][row_in_tile]));
          st_relaxed_gpu(rp.exchange + ((size_t)tm * p.tiles_n + tn) * kBM + row_in_tile, v | kValidBit);
        }

        if (WITH_Y) {
          if (!has_res) {
            if (lane == 0) tma_store_wait_read<0>();
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
            if (cols_ok && row0_warp < p.M) tma_store_2d(&tm_y, y_buf, oc, row0_warp);
            tma_store_commit();
            if (has_res) {
              tma_store_wait_read<0>();
              if (i + 1 < n_my) {
                const int nr = (tm + groups) * kBM + quad * 32;
                mbar_arrive_expect_tx(smem_u32(&res_bar[ew]), kStageBufBytes);
                tma_load_2d(y_buf, &tm_r, cols_ok ? oc : 0, nr < p.M ? nr : 0, smem_u32(&res_bar[ew]));
              }
            }
          }
        }

      }
      if (i >= 1) {
        // -------------------------------------------------------------- pass 2 of tile i - 1
        const int tm = group + (i - 1) * groups;
        const uint32_t buf = (i - 1) & 3;
        const int row0_warp = tm * kBM + quad * 32;
        const int m = row0_warp + lane;
        uint32_t amax_bits = 0u;
        bool valid = true;
#pragma unroll
        for (int t = 0; t < kPrefetchWords; ++t) {
          if (t < p.tiles_n) valid = valid && wait_valid(xrow + (size_t)t * kBM, xw[t], &abort_flag, t_start);
          amax_bits = max(amax_bits, xw[t] & ~kValidBit);
        }
        for (int t = kPrefetchWords; valid && t < p.tiles_n; ++t) {
          uint32_t w = 0u;
          valid = wait_valid(xrow + (size_t)t * kBM, w, &abort_flag, t_start);
          amax_bits = max(amax_bits, w & ~kValidBit);
        }
        if (!__all_sync(0xffffffffu, valid)) { ok = false; break; }
        const float amax = __uint_as_float(amax_bits);
        const ScaleCtx c = make_scale_ctx(amax, rp.qmax_out);
        if (tn == 0 && cpart == 0 && m < p.M) rp.s_out[m] = c.s;
        const uint32_t taddr = tmem_base + buf * BN + ((uint32_t)(quad * 32) << 16) + col;
        uint32_t u[32], w[8];
        tmem_ld_32x32(taddr, u);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tmem_empty_bar[buf]));
        if (rp.pack_out) {
          if (rp.rounding == AQT_ROUND_HALF_UP_FLOOR) codes32<AQT_ROUND_HALF_UP_FLOOR, true>(u, c, rp.qmax_out, w);
          else codes32<AQT_ROUND_NEAREST_EVEN, true>(u, c, rp.qmax_out, w);
        } else {
          if (rp.rounding == AQT_ROUND_HALF_UP_FLOOR) codes32<AQT_ROUND_HALF_UP_FLOOR, false>(u, c, rp.qmax_out, w);
          else codes32<AQT_ROUND_NEAREST_EVEN, false>(u, c, rp.qmax_out, w);
        }
        if (lane == 0) tma_store_wait_read<0>();  // the store that last used the code buffer has read it out
        __syncwarp();
        if (rp.pack_out) {
          // 32 rows of 16 bytes, dense
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(code_buf + lane * 16), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
        } else {
          // 32 rows of 32 bytes under the 32-byte swizzle: 16-byte half h of row r sits at h ^ ((r >> 2) & 1)
          const uint32_t sw = (uint32_t)((lane >> 2) & 1);
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(code_buf + lane * 32 + ((0u ^ sw) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(code_buf + lane * 32 + ((1u ^ sw) << 4)), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (cols_ok && row0_warp < p.M) tma_store_2d(&tm_q, code_buf, rp.pack_out ? oc / 2 : oc, row0_warp);
          tma_store_commit();
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
}

// Bytes of the exchange area (one word per m-tile, n-tile and row).
static size_t requant_exchange_bytes(int64_t M, int64_t N) {
  return round_up((size_t)ceil_div(M, kBM) * (size_t)ceil_div(N, 128) * kBM * 4, 256);
}

// True if this kernel takes the shape.
static bool requant_applies(int64_t M, int64_t N, int64_t K, int act) {
  const int sms = sm_count() > 0 ? sm_count() : 148;
  return M > 0 && ceil_div(K, kBK) <= kWsMaxKBlocks && ceil_div(N, 128) <= sms && (act == AQT_ACT_NONE || act == AQT_ACT_SWISH);
}

template <bool BPACK, bool SMALL, bool WITH_Y>
static int launch_requant_inst(const int8_t* a, const void* b, void* q_out, float* y, int64_t ldy, RequantParams rp,
                               void* exchange, cudaStream_t st) {
  using Cfg = RequantCfg<WITH_Y>;
  GemmParams& p = rp.g;
  p.tiles_m = (int)ceil_div(p.M, kBM);
  p.tiles_n = (int)ceil_div(p.N, Cfg::BN);
  p.k_blocks = (int)ceil_div(p.K, kBK);
  const int sms = sm_count();
  if (sms <= 0) return AQT_ERR_CUDA;
  if (p.k_blocks > kWsMaxKBlocks || p.tiles_n > sms) return AQT_ERR_UNSUPPORTED;
  rp.exchange = reinterpret_cast<uint32_t*>(exchange);
  AQT_RETURN_IF_CUDA(cudaMemsetAsync(exchange, 0, (size_t)p.tiles_m * p.tiles_n * kBM * 4, st));

  CUtensorMap tm_a, tm_b, tm_q, tm_y, tm_r;
  int rc = make_map_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, a, (uint64_t)p.M, (uint64_t)p.K, (uint64_t)p.K, kBM, kBK);
  if (rc != AQT_OK) return rc;
  if (BPACK) rc = make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b, (uint64_t)p.N, (uint64_t)p.K / 2, (uint64_t)p.K / 2, Cfg::BN / 2, 64, 0);
  else rc = make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b, (uint64_t)p.N, (uint64_t)p.K, (uint64_t)p.K, Cfg::BN / 2, kBK);
  if (rc != AQT_OK) return rc;
  if (rp.pack_out) rc = make_map_2d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, q_out, (uint64_t)p.M, (uint64_t)p.N / 2, (uint64_t)p.N / 2, 32, 16, 0);
  else rc = make_map_2d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, q_out, (uint64_t)p.M, (uint64_t)p.N, (uint64_t)p.N, 32, 32, 32);
  if (rc != AQT_OK) return rc;
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
  auto kernel = qgemm_requant_kernel<BPACK, SMALL, WITH_Y>;
  static bool attr_set = false;
  if (!attr_set) {
    AQT_RETURN_IF_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    attr_set = true;
  }
  int groups = sms / p.tiles_n;
  if (groups > p.tiles_m) groups = p.tiles_m;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(groups * p.tiles_n), 1, 1);
  cfg.blockDim = dim3(Cfg::kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // the CTAs wait on one another: all must be resident
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  AQT_RETURN_IF_CUDA(cudaLaunchKernelEx(&cfg, kernel, tm_a, tm_b, tm_q, tm_y, tm_r, rp));
  return AQT_LAUNCH_STATUS();
}

// a: int8 [M, K]; b: int8 [N, K] or (b_packed) nibbles [N, K/2]; y may be null (then no fp32 output
// and no residual).  exchange: requant_exchange_bytes(M, N) bytes.
static int launch_requant(const int8_t* a, const void* b, bool b_packed, void* q_out, float* y, int64_t ldy, const RequantParams& rp,
                          void* exchange, cudaStream_t st) {
  const bool small = rp.g.small_acc != 0;
#define AQT_RQ(BP, SM, WY) launch_requant_inst<BP, SM, WY>(a, b, q_out, y, ldy, rp, exchange, st)
  if (y != nullptr) {
    if (b_packed) return small ? AQT_RQ(true, true, true) : AQT_RQ(true, false, true);
    return small ? AQT_RQ(false, true, true) : AQT_RQ(false, false, true);
  }
  if (b_packed) return small ? AQT_RQ(true, true, false) : AQT_RQ(true, false, false);
  return small ? AQT_RQ(false, true, false) : AQT_RQ(false, false, false);
#undef AQT_RQ
}

}  // namespace aqt
