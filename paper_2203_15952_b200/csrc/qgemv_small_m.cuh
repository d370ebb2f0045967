// Small-batch form of the quantized matmul (M <= 16 rows: streaming / on-device use, where a step
// carries a few frames).  The same arithmetic as the tensor-core kernel -- exact int32
// accumulation of int8 / int4 codes, then z = fma(float(acc) * s_x, s_w, bias), activation,
// residual -- but bound by reading the weights once: 4-bit weights are read packed (half the
// bytes, which is the size / latency argument of Section 4.2 of the paper) and sign-extended in
// registers, activations live in shared memory, products go through dp4a.
//
// One warp per output channel (two channels for GLU: value and gate): each lane takes 16 codes of
// K per step (one 16-byte or 8-byte load, contiguous across the warp), accumulates all rows, and
// a butterfly reduction finishes the sums; lane m then runs the epilogue of row m.
#pragma once

#include "aqt_common.cuh"
#include "pack.cuh"

namespace aqt {

constexpr int kSmallMaxRows = 16;  // measured: from 32 rows on the 128-row tensor-core tile is as fast or faster
constexpr int kSmallMaxK = 6144;  // rows * K bytes of codes must fit shared memory
constexpr int kSmallThreads = 256;

struct SmallParams {
  const void* xq;      // int8 [M, K] or packed [M, K/2]
  const void* wq;      // int8 [N, K] or packed [N, K/2]
  const float* s_x;
  const float* s_w;
  const float* bias;
  const float* residual;
  float* y;
  int32_t* acc_debug;
  int64_t ldr, ldy;
  float residual_scale;
  int s_x_kind, act;
  int M, N, K;
  int a_packed, w_packed;
};

__device__ __forceinline__ float small_sigmoid(float z) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(z * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return r;
}

// 16 weight codes of one channel as four int8x4 words.
template <bool WPACK>
__device__ __forceinline__ void load_w16(const void* wq, int64_t row, int K, int k0, uint32_t (&w)[4]) {
  if (WPACK) {
    const uint2 pk = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint8_t*>(wq) + row * (K / 2) + k0 / 2));
    unpack_word(pk.x, w[0], w[1]);
    unpack_word(pk.y, w[2], w[3]);
  } else {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const int8_t*>(wq) + row * K + k0));
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  }
}

template <int MB, bool WPACK, bool GLU>
__global__ void __launch_bounds__(kSmallThreads) qgemv_small_m_kernel(const SmallParams p) {
  extern __shared__ __align__(16) uint8_t xs[];  // [MB][Kp] activation codes, zero padded
  const int Kp = (p.K + 511) / 512 * 512;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // stage the activation codes (sign-extending 4-bit ones); rows >= M and k >= K are zero
  for (int i = threadIdx.x * 16; i < MB * Kp; i += kSmallThreads * 16) {
    const int m = i / Kp, k = i - m * Kp;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (m < p.M && k < p.K) {
      if (p.a_packed) {
        const uint2 pk = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint8_t*>(p.xq) + (int64_t)m * (p.K / 2) + k / 2));
        unpack_word(pk.x, v.x, v.y);
        unpack_word(pk.y, v.z, v.w);
      } else {
        v = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const int8_t*>(p.xq) + (int64_t)m * p.K + k));
      }
    }
    *reinterpret_cast<uint4*>(xs + i) = v;
  }
  __syncthreads();

  const int channels = GLU ? p.N / 2 : p.N;
  for (int ch = blockIdx.x * (kSmallThreads / 32) + warp; ch < channels; ch += gridDim.x * (kSmallThreads / 32)) {
    int acc0[MB], acc1[GLU ? MB : 1];
#pragma unroll
    for (int m = 0; m < MB; ++m) acc0[m] = 0;
    if (GLU) {
#pragma unroll
      for (int m = 0; m < MB; ++m) acc1[m] = 0;
    }
    for (int k0 = lane * 16; k0 < p.K; k0 += 512) {
      uint32_t w0[4], w1[4];
      load_w16<WPACK>(p.wq, ch, p.K, k0, w0);
      if (GLU) load_w16<WPACK>(p.wq, (int64_t)ch + p.N / 2, p.K, k0, w1);
#pragma unroll
      for (int m = 0; m < MB; ++m) {
        const uint4 x = *reinterpret_cast<const uint4*>(xs + m * Kp + k0);
        acc0[m] = __dp4a((int)x.x, (int)w0[0], acc0[m]);
        acc0[m] = __dp4a((int)x.y, (int)w0[1], acc0[m]);
        acc0[m] = __dp4a((int)x.z, (int)w0[2], acc0[m]);
        acc0[m] = __dp4a((int)x.w, (int)w0[3], acc0[m]);
        if (GLU) {
          acc1[m] = __dp4a((int)x.x, (int)w1[0], acc1[m]);
          acc1[m] = __dp4a((int)x.y, (int)w1[1], acc1[m]);
          acc1[m] = __dp4a((int)x.z, (int)w1[2], acc1[m]);
          acc1[m] = __dp4a((int)x.w, (int)w1[3], acc1[m]);
        }
      }
    }
    // butterfly: every lane ends with every row's full sum; lane m keeps row m
    int mine0 = 0, mine1 = 0;
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      int v = acc0[m];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (lane == m) mine0 = v;
      if (GLU) {
        int g = acc1[m];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) g += __shfl_xor_sync(0xffffffffu, g, off);
        if (lane == m) mine1 = g;
      }
    }
    if (lane < p.M) {
      const int m = lane;
      const float sx = (p.s_x_kind == AQT_SCALE_ROW) ? __ldg(p.s_x + m) : __ldg(p.s_x);
      const float b0 = p.bias != nullptr ? __ldg(p.bias + ch) : 0.0f;
      float a = __fmaf_rn(__fmul_rn(__int2float_rn(mine0), sx), __ldg(p.s_w + ch), b0);
      if (p.acc_debug != nullptr) p.acc_debug[(int64_t)m * p.N + ch] = mine0;
      if (GLU) {
        const int ng = ch + p.N / 2;
        const float b1 = p.bias != nullptr ? __ldg(p.bias + ng) : 0.0f;
        const float zg = __fmaf_rn(__fmul_rn(__int2float_rn(mine1), sx), __ldg(p.s_w + ng), b1);
        if (p.acc_debug != nullptr) p.acc_debug[(int64_t)m * p.N + ng] = mine1;
        a = a * small_sigmoid(zg);
        if (p.act == AQT_ACT_GLU_SWISH) a = a * small_sigmoid(a);
      } else if (p.act == AQT_ACT_SWISH) {
        a = a * small_sigmoid(a);
      }
      if (p.residual != nullptr) a = __fmaf_rn(p.residual_scale, a, __ldg(p.residual + (int64_t)m * p.ldr + ch));
      p.y[(int64_t)m * p.ldy + ch] = a;
    }
  }
}

static bool small_m_applies(int64_t M, int64_t K) {
  const char* lim = tuning_env("AQT_SMALL_M_MAX");  // tuning builds: 0 disables this kernel
  const int64_t max_rows = lim != nullptr ? atoi(lim) : kSmallMaxRows;
  return M >= 1 && M <= max_rows && M <= kSmallMaxRows && K <= kSmallMaxK;
}

template <int MB>
static int launch_small_m_mb(const SmallParams& p, cudaStream_t st) {
  const bool glu = (p.act == AQT_ACT_GLU) || (p.act == AQT_ACT_GLU_SWISH);
  const int Kp = (p.K + 511) / 512 * 512;
  const size_t smem = (size_t)MB * Kp;
  const int channels = glu ? p.N / 2 : p.N;
  const unsigned grid = (unsigned)ceil_div(channels, kSmallThreads / 32);
#define AQT_SMALL_LAUNCH(WP, GL)                                                                                    \
  do {                                                                                                              \
    auto kernel = qgemv_small_m_kernel<MB, WP, GL>;                                                                 \
    static std::atomic<uint64_t> smem_opted_in{0};                                                                  \
    if (smem > 48 * 1024) {                                                                                         \
      const int rc_attr = ensure_dynamic_smem(kernel, MB * kSmallMaxK, smem_opted_in);                              \
      if (rc_attr != AQT_OK) return rc_attr;                                                                        \
    }                                                                                                               \
    kernel<<<grid, kSmallThreads, smem, st>>>(p);                                                                   \
  } while (0)
  if (p.w_packed) {
    if (glu) AQT_SMALL_LAUNCH(true, true); else AQT_SMALL_LAUNCH(true, false);
  } else {
    if (glu) AQT_SMALL_LAUNCH(false, true); else AQT_SMALL_LAUNCH(false, false);
  }
#undef AQT_SMALL_LAUNCH
  return AQT_LAUNCH_STATUS();
}

static int launch_small_m(const SmallParams& p, cudaStream_t st) {
  if (p.M <= 8) return launch_small_m_mb<8>(p, st);
  return launch_small_m_mb<16>(p, st);
}

}  // namespace aqt
