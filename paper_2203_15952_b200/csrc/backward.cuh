// Prepass kernels of the straight-through backward of the quantized linear layer.
//
//   dx[m][k] = sum_n dy[m][n] * s_w[n] * wq[n][k]      dw[n][k] = sum_m dy[m][n] * s_x[m] * xq[m][k]
//   db[n]    = sum_m dy[m][n]
//
// Both products are float contractions against integer codes and run on the float kind of the
// GEMM kernel (qgemm_sm100.cuh), which wants both operands with the contraction index contiguous.
// The kernels here put them in that form: codes transposed, converted to float and multiplied by
// their scale (which varies along the contraction in the backward products, so it cannot stay
// outside the sum as in the forward), and the upstream gradient transposed for dw.
#pragma once

#include "aqt_common.cuh"

namespace aqt {

constexpr int kTrTile = 32;

// codes [R, C] (int8, or nibble pairs along C if packed), scale [R] (or one value if !per_row)
//   -> out [C, ldo] floats, out[c][r] = scale[r] * float(code[r][c]);  columns r in [R, ldo) are zero.
__global__ void __launch_bounds__(256) transpose_scale_codes_kernel(const uint8_t* __restrict__ codes, bool packed,
                                                                    const float* __restrict__ scale, bool per_row, int64_t R,
                                                                    int64_t C, float* __restrict__ out, int64_t ldo) {
  __shared__ float tile[kTrTile][kTrTile + 1];
  const int64_t r0 = (int64_t)blockIdx.y * kTrTile, c0 = (int64_t)blockIdx.x * kTrTile;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int i = ty; i < kTrTile; i += 8) {
    const int64_t r = r0 + i, c = c0 + tx;
    float v = 0.0f;
    if (r < R && c < C) {
      int code;
      if (packed) {
        const uint32_t b = codes[r * (C / 2) + (c >> 1)];
        code = (c & 1) ? ((int)(b << 24) >> 28) : ((int)(b << 28) >> 28);
      } else {
        code = (int)(int8_t)codes[r * C + c];
      }
      v = __fmul_rn(__ldg(scale + (per_row ? r : 0)), (float)code);
    }
    tile[i][tx] = v;
  }
  __syncthreads();
  for (int i = ty; i < kTrTile; i += 8) {
    const int64_t c = c0 + i, r = r0 + tx;
    if (c < C && r < ldo) out[c * ldo + r] = tile[tx][i];
  }
}

// x [R, C] floats with row pitch ldx -> out [C, ldo], out[c][r] = x[r][c]; columns r in [R, ldo) are zero.
__global__ void __launch_bounds__(256) transpose_f32_kernel(const float* __restrict__ x, int64_t ldx, int64_t R, int64_t C,
                                                            float* __restrict__ out, int64_t ldo) {
  __shared__ float tile[kTrTile][kTrTile + 1];
  const int64_t r0 = (int64_t)blockIdx.y * kTrTile, c0 = (int64_t)blockIdx.x * kTrTile;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < kTrTile; i += 8) {
    const int64_t r = r0 + i, c = c0 + tx;
    tile[i][tx] = (r < R && c < C) ? __ldg(x + r * ldx + c) : 0.0f;
  }
  __syncthreads();
  for (int i = ty; i < kTrTile; i += 8) {
    const int64_t c = c0 + i, r = r0 + tx;
    if (c < C && r < ldo) out[c * ldo + r] = tile[tx][i];
  }
}

// Column sums of x [R, C] in a fixed order (the same bits on every run): stage 1 sums the rows of
// one chunk of kColsumChunk rows per block row, top to bottom per thread, then the eight partial
// sums of a column in order; stage 2 adds the chunks' partial sums in order.
constexpr int kColsumChunk = 2048;
__global__ void __launch_bounds__(256) colsum_stage1_kernel(const float* __restrict__ x, int64_t ldx, int64_t R, int64_t C,
                                                            float* __restrict__ partial) {
  __shared__ float acc[8][kTrTile];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t c = (int64_t)blockIdx.x * kTrTile + tx;
  const int64_t r_begin = (int64_t)blockIdx.y * kColsumChunk;
  const int64_t r_end = r_begin + kColsumChunk < R ? r_begin + kColsumChunk : R;
  float s = 0.0f;
  if (c < C)
    for (int64_t r = r_begin + ty; r < r_end; r += 8) s = __fadd_rn(s, __ldg(x + r * ldx + c));
  acc[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && c < C) {
    float t = acc[0][tx];
#pragma unroll
    for (int i = 1; i < 8; ++i) t = __fadd_rn(t, acc[i][tx]);
    partial[(int64_t)blockIdx.y * C + c] = t;
  }
}
__global__ void __launch_bounds__(256) colsum_stage2_kernel(const float* __restrict__ partial, int64_t chunks, int64_t C,
                                                            float* __restrict__ out) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  float t = 0.0f;
  for (int64_t j = 0; j < chunks; ++j) t = __fadd_rn(t, partial[j * C + c]);
  out[c] = t;
}

__global__ void __launch_bounds__(256) fill_f32_kernel(float* __restrict__ p, int64_t n, float v) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

static int launch_transpose_scale_codes(const void* codes, bool packed, const float* scale, bool per_row, int64_t R, int64_t C, float* out,
                                        int64_t ldo, cudaStream_t st) {
  const dim3 grid((unsigned)ceil_div(C, kTrTile), (unsigned)ceil_div(ldo, kTrTile));
  transpose_scale_codes_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const uint8_t*>(codes), packed, scale, per_row, R, C, out, ldo);
  return AQT_LAUNCH_STATUS();
}
static int launch_transpose_f32(const float* x, int64_t ldx, int64_t R, int64_t C, float* out, int64_t ldo, cudaStream_t st) {
  const dim3 grid((unsigned)ceil_div(C, kTrTile), (unsigned)ceil_div(ldo, kTrTile));
  transpose_f32_kernel<<<grid, 256, 0, st>>>(x, ldx, R, C, out, ldo);
  return AQT_LAUNCH_STATUS();
}
static int64_t colsum_chunks(int64_t R) { return ceil_div(R, kColsumChunk); }
static int launch_colsum(const float* x, int64_t ldx, int64_t R, int64_t C, float* partial, float* out, cudaStream_t st) {
  const int64_t chunks = colsum_chunks(R);
  colsum_stage1_kernel<<<dim3((unsigned)ceil_div(C, kTrTile), (unsigned)chunks), 256, 0, st>>>(x, ldx, R, C, partial);
  int rc = AQT_LAUNCH_STATUS();
  if (rc != AQT_OK) return rc;
  colsum_stage2_kernel<<<(unsigned)ceil_div(C, 256), 256, 0, st>>>(partial, chunks, C, out);
  return AQT_LAUNCH_STATUS();
}
static int launch_fill_f32(float* p, int64_t n, float v, cudaStream_t st) {
  fill_f32_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(p, n, v);
  return AQT_LAUNCH_STATUS();
}

}  // namespace aqt
