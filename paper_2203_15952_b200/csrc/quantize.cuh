// Activation / weight quantizer kernels: Fig. 2 of the paper (abs-max over the reduced axis,
// scale = amax / qmax, divide_no_nan, round, int8 container) and its int4 form (Section 2.2).
// HBM-bound: one read of fp32 x, one write of codes and scales.
#pragma once

#include "aqt_common.cuh"

namespace aqt {

constexpr int kQuantThreads = 256;
constexpr int kQuantMaxVec = 4;  // float4 loads held in registers per thread (16 elements)

// Pack four codes (sign-extended ints) into the output word: int8 container (4 bytes) or nibbles
// (2 bytes).  Byte permutes take the low byte of each code.
__device__ __forceinline__ uint32_t pack4_i8(int a, int b, int c, int d) {
  const uint32_t lo = __byte_perm((uint32_t)a, (uint32_t)b, 0x0040);  // a.b0, b.b0
  const uint32_t hi = __byte_perm((uint32_t)c, (uint32_t)d, 0x0040);  // c.b0, d.b0
  return __byte_perm(lo, hi, 0x5410);
}
__device__ __forceinline__ uint32_t pack4_i4(int a, int b, int c, int d) {
  const uint32_t x = pack4_i8(a, b, c, d) & 0x0F0F0F0Fu;
  const uint32_t y = x | (x >> 4);         // byte 0 = n0 | n1 << 4, byte 2 = n2 | n3 << 4
  return __byte_perm(y, 0u, 0x4420) & 0xFFFFu;
}

// Four elements of a row whose scale constants are known, fast path of quantize_elem: the
// correctly rounded quotient by one multiply and two FMAs, then one conversion.  No clip: with
// abs-max scaling |x / s| <= qmax (1 + 2^-23), which every rounding rule maps inside +-qmax; the
// clip only matters for the subnormal scales that never take this path.
template <int ROUNDING>
__device__ __forceinline__ int quantize_fast(float x, float s, float r) {
  const float q0 = __fmul_rn(x, r);
  const float e = __fmaf_rn(-q0, s, x);
  const float v = __fmaf_rn(e, r, q0);
  if (ROUNDING == AQT_ROUND_HALF_UP_FLOOR) return __float2int_rd(__fadd_rn(v, 0.5f));
  return __float2int_rn(v);
}

// Per-row quantizer, row held in registers.  G threads cooperate on one row (G a power of two,
// 32 <= G <= 256); each thread owns up to kQuantMaxVec float4s, strided by G so that every load
// and store instruction of a warp is contiguous.  Requires cols % 4 == 0, ld % 4 == 0, x 16-byte
// aligned, cols <= 16 * G.
template <int G, int ROUNDING, bool PACK>
__global__ void __launch_bounds__(kQuantThreads) quantize_rows_reg_kernel(
    const float* __restrict__ x, int64_t rows, int cols, int64_t ld, int qmax, void* __restrict__ q_out,
    float* __restrict__ scale_out) {
  constexpr int ROWS_PER_CTA = kQuantThreads / G;
  constexpr int WARPS_PER_ROW = G / 32;
  __shared__ float warp_max[kQuantThreads / 32];

  grid_dependency_wait();
  const int t = threadIdx.x % G;
  const int r_in_cta = threadIdx.x / G;
  const int64_t row = (int64_t)blockIdx.x * ROWS_PER_CTA + r_in_cta;
  const bool live = row < rows;
  const int nvec = cols >> 2;
  const float4* xrow = reinterpret_cast<const float4*>(x + (live ? row : 0) * ld);

  float4 v[kQuantMaxVec];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < kQuantMaxVec; ++i) {
    const int idx = t + i * G;
    v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live && idx < nvec) v[i] = __ldg(xrow + idx);
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v[i].x), fabsf(v[i].y)), fmaxf(fabsf(v[i].z), fabsf(v[i].w))));
  }
  grid_dependents_launch();  // this CTA's loads are in flight; it has little left to do
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if (WARPS_PER_ROW > 1) {
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) warp_max[warp] = amax;
    __syncthreads();
    const int w0 = r_in_cta * WARPS_PER_ROW;
#pragma unroll
    for (int w = 0; w < WARPS_PER_ROW; ++w) amax = fmaxf(amax, warp_max[w0 + w]);
  }
  if (!live) return;

  const ScaleCtx c = make_scale_ctx(amax, qmax);
  if (t == 0) scale_out[row] = c.s;

#pragma unroll
  for (int i = 0; i < kQuantMaxVec; ++i) {
    const int idx = t + i * G;
    if (idx < nvec) {
      int a, b, cc, d;
      if (c.fast) {  // uniform over the row
        a = quantize_fast<ROUNDING>(v[i].x, c.s, c.r);
        b = quantize_fast<ROUNDING>(v[i].y, c.s, c.r);
        cc = quantize_fast<ROUNDING>(v[i].z, c.s, c.r);
        d = quantize_fast<ROUNDING>(v[i].w, c.s, c.r);
      } else {
        a = quantize_elem<ROUNDING>(v[i].x, c, qmax);
        b = quantize_elem<ROUNDING>(v[i].y, c, qmax);
        cc = quantize_elem<ROUNDING>(v[i].z, c, qmax);
        d = quantize_elem<ROUNDING>(v[i].w, c, qmax);
      }
      // one output word per float4: 2 bytes of nibbles or 4 bytes of int8 codes
      if (PACK) {
        reinterpret_cast<uint16_t*>(q_out)[row * (int64_t)nvec + idx] = (uint16_t)pack4_i4(a, b, cc, d);
      } else {
        reinterpret_cast<uint32_t*>(q_out)[row * (int64_t)nvec + idx] = pack4_i8(a, b, cc, d);
      }
    }
  }
}

// Per-row quantizer for any cols / ld / alignment: one CTA per row, two passes over the row
// (the second pass re-reads what the first just brought into L1/L2).
template <int ROUNDING, bool PACK>
__global__ void __launch_bounds__(kQuantThreads) quantize_rows_generic_kernel(
    const float* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, int qmax, void* __restrict__ q_out,
    float* __restrict__ scale_out) {
  __shared__ float warp_max[kQuantThreads / 32];
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float* xr = x + row * ld;
    float amax = 0.0f;
    for (int64_t j = threadIdx.x; j < cols; j += kQuantThreads) amax = fmaxf(amax, fabsf(xr[j]));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
    __syncthreads();  // warp_max of the previous row is no longer read
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kQuantThreads / 32; ++w) amax = fmaxf(amax, warp_max[w]);
    const ScaleCtx c = make_scale_ctx(amax, qmax);
    if (threadIdx.x == 0) scale_out[row] = c.s;
    if (PACK) {
      uint8_t* qr = reinterpret_cast<uint8_t*>(q_out) + row * (cols / 2);
      for (int64_t j = threadIdx.x; j < cols / 2; j += kQuantThreads) {
        const int lo = quantize_elem<ROUNDING>(xr[2 * j], c, qmax);
        const int hi = quantize_elem<ROUNDING>(xr[2 * j + 1], c, qmax);
        qr[j] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
      }
    } else {
      int8_t* qr = reinterpret_cast<int8_t*>(q_out) + row * cols;
      for (int64_t j = threadIdx.x; j < cols; j += kQuantThreads) qr[j] = (int8_t)quantize_elem<ROUNDING>(xr[j], c, qmax);
    }
  }
}

// abs-max accumulation for the column and tensor axes.  Non-negative floats order like their
// bit patterns, so atomicMax on the unsigned view is a float max.  amax_bits must be zeroed
// before the launch; it has `cols` slots (per_col) or one.
__global__ void __launch_bounds__(kQuantThreads) absmax_accumulate_kernel(
    const float* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, bool per_col, unsigned* __restrict__ amax_bits) {
  if (per_col) {
    // thread <-> column (coalesced across the warp), CTA.y strides over row chunks
    const int64_t col = (int64_t)blockIdx.x * kQuantThreads + threadIdx.x;
    if (col >= cols) return;
    float amax = 0.0f;
    for (int64_t r = blockIdx.y; r < rows; r += gridDim.y) amax = fmaxf(amax, fabsf(x[r * ld + col]));
    atomicMax(amax_bits + col, __float_as_uint(amax));
  } else {
    __shared__ float warp_max[kQuantThreads / 32];
    float amax = 0.0f;
    const int64_t total = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * kQuantThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kQuantThreads) {
      const int64_t r = i / cols, j = i - r * cols;
      amax = fmaxf(amax, fabsf(x[r * ld + j]));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < kQuantThreads / 32; ++w) amax = fmaxf(amax, warp_max[w]);
      atomicMax(amax_bits, __float_as_uint(amax));
    }
  }
}

// amax -> scale in place (scale = amax / qmax, IEEE division).
__global__ void finalize_scales_kernel(float* __restrict__ scale, int64_t n, int qmax) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) scale[i] = __fdiv_rn(scale[i], (float)qmax);
}

// Element-wise quantization against scales that are already final (column or tensor axis).
// One thread per pair of adjacent columns so that packed output needs no cross-thread exchange.
template <int ROUNDING, bool PACK>
__global__ void __launch_bounds__(kQuantThreads) quantize_with_scales_kernel(
    const float* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, bool per_col, int qmax,
    const float* __restrict__ scale, void* __restrict__ q_out) {
  const int64_t pairs_per_row = (cols + 1) / 2;
  const int64_t total = rows * pairs_per_row;
  for (int64_t i = (int64_t)blockIdx.x * kQuantThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kQuantThreads) {
    const int64_t r = i / pairs_per_row, p = i - r * pairs_per_row;
    const int64_t j0 = 2 * p, j1 = 2 * p + 1;
    // the scale is already divided; rebuild the per-scale constants from it
    ScaleCtx c0, c1;
    c0.s = scale[per_col ? j0 : 0];
    c0.fast = (c0.s >= 1.2e-20f) && (c0.s <= 8.0e15f);
    c0.r = c0.fast ? __frcp_rn(c0.s) : 0.0f;
    const int a = quantize_elem<ROUNDING>(x[r * ld + j0], c0, qmax);
    int b = 0;
    if (j1 < cols) {
      c1 = c0;
      if (per_col) {
        c1.s = scale[j1];
        c1.fast = (c1.s >= 1.2e-20f) && (c1.s <= 8.0e15f);
        c1.r = c1.fast ? __frcp_rn(c1.s) : 0.0f;
      }
      b = quantize_elem<ROUNDING>(x[r * ld + j1], c1, qmax);
    }
    if (PACK) {
      reinterpret_cast<uint8_t*>(q_out)[r * (cols / 2) + p] = (uint8_t)((a & 0xF) | ((b & 0xF) << 4));
    } else {
      int8_t* q = reinterpret_cast<int8_t*>(q_out) + r * cols;
      q[j0] = (int8_t)a;
      if (j1 < cols) q[j1] = (int8_t)b;
    }
  }
}

// Whole-tensor scale for small tensors in one launch: one CTA finds the abs-max, forms the scale
// and quantizes (the tensor is re-read from L1/L2).  Replaces the four-launch path below where
// launch latency, not bandwidth, is the cost (e.g. a [64, 256] activation).
constexpr int kSmallTensorElems = 1 << 16;
template <int ROUNDING, bool PACK>
__global__ void __launch_bounds__(1024) quantize_tensor_small_kernel(const float* __restrict__ x, int rows, int cols, int64_t ld,
                                                                      int qmax, void* __restrict__ q_out,
                                                                      float* __restrict__ scale_out) {
  __shared__ float warp_max[32];
  const int total = rows * cols;
  // dense, aligned tensors of up to 16 K elements stay in registers: all loads are issued at once
  const bool in_regs = (ld == cols) && (total % 4 == 0) && (total <= 4 * 4 * 1024) &&
                       ((reinterpret_cast<uintptr_t>(x) & 15) == 0) && ((reinterpret_cast<uintptr_t>(q_out) & 3) == 0);
  float4 v[4];
  float amax = 0.0f;
  if (in_regs) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = threadIdx.x + i * 1024;
      v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (idx < total / 4) v[i] = __ldg(reinterpret_cast<const float4*>(x) + idx);
      amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v[i].x), fabsf(v[i].y)), fmaxf(fabsf(v[i].z), fabsf(v[i].w))));
    }
  } else {
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
      const int r = i / cols, j = i - r * cols;
      amax = fmaxf(amax, fabsf(x[(int64_t)r * ld + j]));
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = 0.0f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) amax = fmaxf(amax, warp_max[w]);
  const ScaleCtx c = make_scale_ctx(amax, qmax);
  if (threadIdx.x == 0) scale_out[0] = c.s;
  if (in_regs) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = threadIdx.x + i * 1024;
      if (idx < total / 4) {
        const int a = quantize_elem<ROUNDING>(v[i].x, c, qmax), b = quantize_elem<ROUNDING>(v[i].y, c, qmax);
        const int cc = quantize_elem<ROUNDING>(v[i].z, c, qmax), d = quantize_elem<ROUNDING>(v[i].w, c, qmax);
        if (PACK) reinterpret_cast<uint16_t*>(q_out)[idx] = (uint16_t)pack4_i4(a, b, cc, d);
        else reinterpret_cast<uint32_t*>(q_out)[idx] = pack4_i8(a, b, cc, d);
      }
    }
    return;
  }
  const int pairs_per_row = (cols + 1) / 2;
  for (int i = threadIdx.x; i < rows * pairs_per_row; i += blockDim.x) {
    const int r = i / pairs_per_row, p = i - r * pairs_per_row;
    const int j0 = 2 * p, j1 = 2 * p + 1;
    const int a = quantize_elem<ROUNDING>(x[(int64_t)r * ld + j0], c, qmax);
    const int b = j1 < cols ? quantize_elem<ROUNDING>(x[(int64_t)r * ld + j1], c, qmax) : 0;
    if (PACK) {
      reinterpret_cast<uint8_t*>(q_out)[(int64_t)r * (cols / 2) + p] = (uint8_t)((a & 0xF) | ((b & 0xF) << 4));
    } else {
      int8_t* q = reinterpret_cast<int8_t*>(q_out) + (int64_t)r * cols;
      q[j0] = (int8_t)a;
      if (j1 < cols) q[j1] = (int8_t)b;
    }
  }
}

template <int ROUNDING, bool PACK>
static int launch_quantize_rows(const float* x, int64_t rows, int64_t cols, int64_t ld, int qmax, void* q_out,
                                float* scale_out, cudaStream_t st) {
  const bool vec_ok = (cols % 4 == 0) && (ld % 4 == 0) && is_aligned(x, 16) && cols <= 16 * 256 &&
                      is_aligned(q_out, 4);
  if (vec_ok) {
    const int nvec = (int)(cols / 4);
#define AQT_LAUNCH_ROWS(G)                                                                                   \
  do {                                                                                                       \
    const int64_t grid = ceil_div(rows, kQuantThreads / G);                                                  \
    const int rc_launch = launch_pdl(quantize_rows_reg_kernel<G, ROUNDING, PACK>, dim3((unsigned)grid, 1, 1),       \
                                     dim3(kQuantThreads, 1, 1), 0, st, 1, x, rows, (int)cols, ld, qmax, q_out, scale_out); \
    if (rc_launch != AQT_OK) return rc_launch;                                                               \
  } while (0)
    if (nvec <= 32 * kQuantMaxVec) AQT_LAUNCH_ROWS(32);
    else if (nvec <= 64 * kQuantMaxVec) AQT_LAUNCH_ROWS(64);
    else if (nvec <= 128 * kQuantMaxVec) AQT_LAUNCH_ROWS(128);
    else AQT_LAUNCH_ROWS(256);
#undef AQT_LAUNCH_ROWS
  } else {
    const int64_t grid = rows < 148 * 16 ? rows : 148 * 16;
    quantize_rows_generic_kernel<ROUNDING, PACK><<<(unsigned)grid, kQuantThreads, 0, st>>>(x, rows, cols, ld, qmax, q_out, scale_out);
  }
  return AQT_LAUNCH_STATUS();
}

template <int ROUNDING, bool PACK>
static int launch_quantize_axis(const float* x, int64_t rows, int64_t cols, int64_t ld, int qmax, int axis, void* q_out,
                                float* scale_out, cudaStream_t st) {
  if (axis == AQT_AXIS_ROW) return launch_quantize_rows<ROUNDING, PACK>(x, rows, cols, ld, qmax, q_out, scale_out, st);
  const bool per_col = axis == AQT_AXIS_COL;
  if (!per_col && rows * cols <= kSmallTensorElems) {
    quantize_tensor_small_kernel<ROUNDING, PACK><<<1, 1024, 0, st>>>(x, (int)rows, (int)cols, ld, qmax, q_out, scale_out);
    return AQT_LAUNCH_STATUS();
  }
  const int64_t n_scale = per_col ? cols : 1;
  AQT_RETURN_IF_CUDA(cudaMemsetAsync(scale_out, 0, (size_t)n_scale * sizeof(float), st));
  if (per_col) {
    dim3 grid((unsigned)ceil_div(cols, kQuantThreads), (unsigned)(rows < 64 ? rows : 64));
    absmax_accumulate_kernel<<<grid, kQuantThreads, 0, st>>>(x, rows, cols, ld, true, reinterpret_cast<unsigned*>(scale_out));
  } else {
    const int64_t want = ceil_div(rows * cols, kQuantThreads * 8);
    const unsigned grid = (unsigned)(want < 1 ? 1 : (want > 148 * 8 ? 148 * 8 : want));
    absmax_accumulate_kernel<<<grid, kQuantThreads, 0, st>>>(x, rows, cols, ld, false, reinterpret_cast<unsigned*>(scale_out));
  }
  finalize_scales_kernel<<<(unsigned)ceil_div(n_scale, 256), 256, 0, st>>>(scale_out, n_scale, qmax);
  const int64_t pairs = rows * ((cols + 1) / 2);
  const int64_t want = ceil_div(pairs, kQuantThreads * 4);
  const unsigned grid = (unsigned)(want < 1 ? 1 : (want > 148 * 16 ? 148 * 16 : want));
  quantize_with_scales_kernel<ROUNDING, PACK><<<grid, kQuantThreads, 0, st>>>(x, rows, cols, ld, per_col, qmax, scale_out, q_out);
  return AQT_LAUNCH_STATUS();
}

}  // namespace aqt
