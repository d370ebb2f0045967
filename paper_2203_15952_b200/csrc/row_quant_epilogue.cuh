// What the matmul kernels share when their epilogue quantizes the output rows (Fig. 2 of the paper
// applied to u before it leaves the SM): writing u back to tensor memory, the codes of a chunk of
// a row once its scale is known, and the tagged words through which CTAs exchange row maxima.
#pragma once

#include <atomic>

#include "aqt_common.cuh"

namespace aqt {

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

// A call's tag mixed with a generation count: distinct generations of one call give distinct values.
__device__ __forceinline__ uint32_t mix_tag(uint32_t call_tag, uint32_t generation) {
  uint32_t x = call_tag ^ (generation * 0x9E3779B1u);
  x ^= x >> 16;
  x *= 0x7FEB352Du;
  x ^= x >> 15;
  return x;
}

__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Two exchange words (each read as one indivisible 64-bit value).
__device__ __forceinline__ ulonglong2 ld_relaxed_gpu_2x64(const uint64_t* p) {
  ulonglong2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_gpu_64(uint64_t* p, uint64_t v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}


// Codes of two values whose row scale constants are known (fast path of the quantizer: the
// correctly rounded quotient by one multiply and two fused multiply-adds).  Rounding by adding
// 1.5 * 2^23: the sum's low mantissa bits are the integer in two's complement, so the code's
// byte is the low byte of the sum's bit pattern.  Nearest-even is the add's own rounding; the
// figure's floor(v + 0.5) is the binary32 add of 0.5 followed by an add rounded towards minus
// infinity.  Exact for |v| < 2^22; here |v| <= 127 (1 + 2^-23).
template <int ROUNDING>
__device__ __forceinline__ float2 code_bits2(float2 x, float2 s_neg, float2 r) {
  const float2 q0 = __fmul2_rn(x, r);
  const float2 e = __ffma2_rn(q0, s_neg, x);  // x - q0 s, exact
  const float2 v = __ffma2_rn(e, r, q0);
  const float2 magic = make_float2(12582912.0f, 12582912.0f);
  if (ROUNDING == AQT_ROUND_HALF_UP_FLOOR) return __fadd2_rd(__fadd2_rn(v, make_float2(0.5f, 0.5f)), magic);
  return __fadd2_rn(v, magic);
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

// NV (32 or 16) values of one row -> NV / 4 words of int8 codes (PACK: NV / 8 words of nibbles).
template <int ROUNDING, bool PACK, int NV>
__device__ __forceinline__ void codes_of(const uint32_t (&u)[NV], const ScaleCtx& c, int qmax, uint32_t (&w)[NV / 4]) {
  if (c.fast) {
    const float2 s_neg = make_float2(-c.s, -c.s), r2 = make_float2(c.r, c.r);
#pragma unroll
    for (int j = 0; j < NV / 4; ++j) {
      const float2 c01 = code_bits2<ROUNDING>(make_float2(__uint_as_float(u[4 * j]), __uint_as_float(u[4 * j + 1])), s_neg, r2);
      const float2 c23 = code_bits2<ROUNDING>(make_float2(__uint_as_float(u[4 * j + 2]), __uint_as_float(u[4 * j + 3])), s_neg, r2);
      w[j] = low_bytes(__float_as_uint(c01.x), __float_as_uint(c01.y), __float_as_uint(c23.x), __float_as_uint(c23.y));
    }
  } else {
#pragma unroll
    for (int j = 0; j < NV / 4; ++j)
      w[j] = low_bytes((uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j]), c, qmax),
                       (uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j + 1]), c, qmax),
                       (uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j + 2]), c, qmax),
                       (uint32_t)quantize_elem<ROUNDING>(__uint_as_float(u[4 * j + 3]), c, qmax));
  }
  if (PACK) {
#pragma unroll
    for (int j = 0; j < NV / 8; ++j) w[j] = nibbles_of(w[2 * j], w[2 * j + 1]);
  }
}


// A tag no earlier call of this process has used: a counter run through a bijection of the 32-bit
// integers, so that consecutive tags share no pattern with small integers or with one another.  A
// word of the exchange area counts only if its upper half equals the call's tag mixed with the
// group's generation counter (see the kernel), so the area needs no clearing: whatever another call
// or an earlier execution of this call left there carries another value.  Memory that never held
// exchange words passes for valid with probability 2^-32 per word.
static uint32_t next_launch_tag() {
  static std::atomic<uint32_t> counter{0};
  uint32_t x = counter.fetch_add(1, std::memory_order_relaxed) + 1u;
  x ^= x >> 16;
  x *= 0x7FEB352Du;
  x ^= x >> 15;
  x *= 0x846CA68Bu;
  x ^= x >> 16;
  return x != 0u ? x : 0x9E3779B9u;  // zero marks a wiped word
}

constexpr int kMaxGroups = 256;  // at most one group per SM


}  // namespace aqt
