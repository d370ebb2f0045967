// 4-bit storage kernels: two two's-complement nibbles per byte, even element in the low nibble.
// Rows are dense, so a [rows, cols] tensor with even cols is one flat stream of byte pairs.
#pragma once

#include "aqt_common.cuh"

namespace aqt {

// Sign-extend the low nibble of each of the four bytes of x (high nibbles must be zero):
// a set bit 3 (0x08) times 0x1E gives 0xF0 in the same byte and never carries into the next.
__device__ __forceinline__ uint32_t sext_nibbles_in_bytes(uint32_t x) { return x | ((x & 0x08080808u) * 0x1Eu); }

// Four packed bytes -> eight int8 codes in element order (two 32-bit words).
__device__ __forceinline__ void unpack_word(uint32_t w, uint32_t& out0, uint32_t& out1) {
  const uint32_t lo = sext_nibbles_in_bytes(w & 0x0F0F0F0Fu);
  const uint32_t hi = sext_nibbles_in_bytes((w >> 4) & 0x0F0F0F0Fu);
  out0 = __byte_perm(lo, hi, 0x5140);  // l0 h0 l1 h1
  out1 = __byte_perm(lo, hi, 0x7362);  // l2 h2 l3 h3
}

// Eight int8 codes (two words, element order) -> four packed bytes.
__device__ __forceinline__ uint32_t pack_words(uint32_t w0, uint32_t w1) {
  const uint32_t t0 = (w0 & 0x000F000Fu) | (((w0 >> 8) & 0x000F000Fu) << 4);  // bytes 0 and 2 hold the pairs
  const uint32_t t1 = (w1 & 0x000F000Fu) | (((w1 >> 8) & 0x000F000Fu) << 4);
  return __byte_perm(t0, t1, 0x6420);
}

// n_bytes packed bytes -> 2 * n_bytes codes.  vec path: 8 packed bytes per thread per step.
__global__ void __launch_bounds__(256) unpack_int4_kernel(const uint8_t* __restrict__ packed, int64_t n_bytes,
                                                          int8_t* __restrict__ q, bool vec) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (vec) {
    const int64_t n8 = n_bytes >> 3;
    const uint2* src = reinterpret_cast<const uint2*>(packed);
    uint4* dst = reinterpret_cast<uint4*>(q);
    for (int64_t i = tid; i < n8; i += stride) {
      const uint2 w = __ldg(src + i);
      uint4 o;
      unpack_word(w.x, o.x, o.y);
      unpack_word(w.y, o.z, o.w);
      dst[i] = o;
    }
    for (int64_t i = (n8 << 3) + tid; i < n_bytes; i += stride) {
      const uint32_t b = packed[i];
      q[2 * i] = (int8_t)((int)(b << 28) >> 28);
      q[2 * i + 1] = (int8_t)((int)(b << 24) >> 28);
    }
  } else {
    for (int64_t i = tid; i < n_bytes; i += stride) {
      const uint32_t b = packed[i];
      q[2 * i] = (int8_t)((int)(b << 28) >> 28);
      q[2 * i + 1] = (int8_t)((int)(b << 24) >> 28);
    }
  }
}

__global__ void __launch_bounds__(256) pack_int4_kernel(const int8_t* __restrict__ q, int64_t n_bytes,
                                                        uint8_t* __restrict__ packed, bool vec) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (vec) {
    const int64_t n8 = n_bytes >> 3;
    const uint4* src = reinterpret_cast<const uint4*>(q);
    uint2* dst = reinterpret_cast<uint2*>(packed);
    for (int64_t i = tid; i < n8; i += stride) {
      const uint4 w = __ldg(src + i);
      dst[i] = make_uint2(pack_words(w.x, w.y), pack_words(w.z, w.w));
    }
    for (int64_t i = (n8 << 3) + tid; i < n_bytes; i += stride)
      packed[i] = (uint8_t)((q[2 * i] & 0xF) | ((q[2 * i + 1] & 0xF) << 4));
  } else {
    for (int64_t i = tid; i < n_bytes; i += stride)
      packed[i] = (uint8_t)((q[2 * i] & 0xF) | ((q[2 * i + 1] & 0xF) << 4));
  }
}

// Weight codes -> binary32 values of the same integers (exact; every code has at most 7
// significant bits).  The float matmul of the weight-only layer reads these.  n codes, a multiple
// of 4: dense int8, or nibble pairs if `packed`.  Four codes per thread and step.
__global__ void __launch_bounds__(256) codes_to_float_kernel(const uint8_t* __restrict__ codes, bool packed, int64_t n,
                                                             float* __restrict__ out) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < (n >> 2); i += stride) {
    uint32_t w;
    if (packed) {
      uint32_t o1;
      unpack_word((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(codes) + i), w, o1);
    } else {
      w = __ldg(reinterpret_cast<const uint32_t*>(codes) + i);
    }
    float4 f;
    f.x = (float)(int8_t)(w & 0xFF);
    f.y = (float)(int8_t)((w >> 8) & 0xFF);
    f.z = (float)(int8_t)((w >> 16) & 0xFF);
    f.w = (float)(int8_t)(w >> 24);
    reinterpret_cast<float4*>(out)[i] = f;
  }
}

// Two-term split of binary32 activations for the float matmul: hi = x with its lower thirteen
// fraction bits cleared (a tf32 value), lo = x - hi (exact).  Row m of the output holds
// [hi(x[m][0..K)) | lo(x[m][0..K))], so that one matmul over 2K against the weights repeated twice
// sums x . w with about twenty-one significant bits per activation.  K % 4 == 0, ldx % 4 == 0.
__global__ void __launch_bounds__(256) split_hi_lo_kernel(const float* __restrict__ x, int64_t ldx, int64_t M, int64_t K,
                                                          float* __restrict__ out) {
  const int64_t k4 = K >> 2, total = M * k4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t m = i / k4, c = i - m * k4;
    const float4 v = __ldg(reinterpret_cast<const float4*>(x + m * ldx) + c);
    float4 hi, lo;
    hi.x = __uint_as_float(__float_as_uint(v.x) & 0xFFFFE000u);
    hi.y = __uint_as_float(__float_as_uint(v.y) & 0xFFFFE000u);
    hi.z = __uint_as_float(__float_as_uint(v.z) & 0xFFFFE000u);
    hi.w = __uint_as_float(__float_as_uint(v.w) & 0xFFFFE000u);
    lo.x = __fsub_rn(v.x, hi.x);
    lo.y = __fsub_rn(v.y, hi.y);
    lo.z = __fsub_rn(v.z, hi.z);
    lo.w = __fsub_rn(v.w, hi.w);
    float4* row = reinterpret_cast<float4*>(out + m * 2 * K);
    row[c] = hi;
    row[k4 + c] = lo;
  }
}

// The weight codes as floats, each row written twice: out [rows, 2K] = [w | w].
__global__ void __launch_bounds__(256) codes_to_float_twice_kernel(const uint8_t* __restrict__ codes, bool packed, int64_t rows,
                                                                   int64_t K, float* __restrict__ out) {
  const int64_t k4 = K >> 2, total = rows * k4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t r = i / k4, c = i - r * k4;
    uint32_t w;
    if (packed) {
      uint32_t o1;
      unpack_word((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(codes) + i), w, o1);
    } else {
      w = __ldg(reinterpret_cast<const uint32_t*>(codes) + i);
    }
    float4 f;
    f.x = (float)(int8_t)(w & 0xFF);
    f.y = (float)(int8_t)((w >> 8) & 0xFF);
    f.z = (float)(int8_t)((w >> 16) & 0xFF);
    f.w = (float)(int8_t)(w >> 24);
    float4* row = reinterpret_cast<float4*>(out + r * 2 * K);
    row[c] = f;
    row[k4 + c] = f;
  }
}

static unsigned flat_grid(int64_t work_items) {
  const int64_t want = ceil_div(work_items, 256);
  return (unsigned)(want < 1 ? 1 : (want > 148 * 32 ? 148 * 32 : want));
}

static int launch_unpack_int4(const uint8_t* packed, int64_t n_bytes, int8_t* q, cudaStream_t st) {
  const bool vec = is_aligned(packed, 8) && is_aligned(q, 16);
  unpack_int4_kernel<<<flat_grid(vec ? n_bytes / 8 + 8 : n_bytes), 256, 0, st>>>(packed, n_bytes, q, vec);
  return AQT_LAUNCH_STATUS();
}

// codes: int8 [n] or packed nibbles [n / 2], 4-byte (2-byte if packed) aligned; out: float [n], 16-byte aligned; n % 4 == 0.
static int launch_codes_to_float(const void* codes, bool packed, int64_t n, float* out, cudaStream_t st) {
  codes_to_float_kernel<<<flat_grid(n / 4), 256, 0, st>>>(reinterpret_cast<const uint8_t*>(codes), packed, n, out);
  return AQT_LAUNCH_STATUS();
}

static int launch_split_hi_lo(const float* x, int64_t ldx, int64_t M, int64_t K, float* out, cudaStream_t st) {
  split_hi_lo_kernel<<<flat_grid(M * K / 4), 256, 0, st>>>(x, ldx, M, K, out);
  return AQT_LAUNCH_STATUS();
}
static int launch_codes_to_float_twice(const void* codes, bool packed, int64_t rows, int64_t K, float* out, cudaStream_t st) {
  codes_to_float_twice_kernel<<<flat_grid(rows * K / 4), 256, 0, st>>>(reinterpret_cast<const uint8_t*>(codes), packed, rows, K, out);
  return AQT_LAUNCH_STATUS();
}

static int launch_pack_int4(const int8_t* q, int64_t n_bytes, uint8_t* packed, cudaStream_t st) {
  const bool vec = is_aligned(packed, 8) && is_aligned(q, 16);
  pack_int4_kernel<<<flat_grid(vec ? n_bytes / 8 + 8 : n_bytes), 256, 0, st>>>(q, n_bytes, packed, vec);
  return AQT_LAUNCH_STATUS();
}

}  // namespace aqt
