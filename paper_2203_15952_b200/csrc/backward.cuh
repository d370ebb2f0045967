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
#include "pack.cuh"

namespace aqt {

constexpr int kTrTile = 32;

// Output layout of both transposes: the input's row index r (the contraction index of the matmul
// that follows) is cut into chunks of `chunk` rows; chunk s of input column c goes to output row
// s * rows_out + c, so that the chunks form a stack of [rows_out, chunk] matrices:
//   out[(r / chunk * rows_out + c) * chunk + r % chunk] = value(r, c),  zero for r in [R, r_pad).
// With one chunk (chunk = r_pad >= R) this is the plain transpose [C, chunk].  With several, chunk
// is a multiple of the tile height, so a tile lies in one chunk.  Rows c in [C, rows_out) of a
// batch are not written (their products land in output rows or columns nobody reads).
// A block moves a tile of kTrRows input rows x 32 input columns through shared memory: sixteen
// independent loads per thread, then 512-byte runs of the output.
constexpr int kTrRows = 128;

// codes [R, C] (int8, or nibble pairs along C if packed), scale [R] (or one value if !per_row)
//   -> value(r, c) = scale[r] * float(code[r][c]) in the layout above.
__global__ void __launch_bounds__(256) transpose_scale_codes_kernel(const uint8_t* __restrict__ codes, bool packed,
                                                                    const float* __restrict__ scale, bool per_row, int64_t R,
                                                                    int64_t C, float* __restrict__ out, int64_t r_pad, int64_t chunk,
                                                                    int64_t rows_out) {
  __shared__ float tile[kTrRows][kTrTile + 1];
  const int64_t r0 = (int64_t)blockIdx.y * kTrRows, c0 = (int64_t)blockIdx.x * kTrTile;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  // load: four codes (one 32-bit word, or two packed bytes) per thread and step; eight threads cover a row of the tile
#pragma unroll
  for (int j = 0; j < kTrRows * kTrTile / 4 / 256; ++j) {
    const int w = threadIdx.x + 256 * j;
    const int i = w >> 3, cw = w & 7;
    const int64_t r = r0 + i, c = c0 + 4 * cw;  // C is a multiple of 4, so a word is inside the row or outside it
    float v0 = 0.0f, v1 = 0.0f, v2 = 0.0f, v3 = 0.0f;
    if (r < R && c < C) {
      uint32_t word;
      if (packed) {
        uint32_t hi;
        unpack_word((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(codes + r * (C / 2) + (c >> 1))), word, hi);
      } else {
        word = __ldg(reinterpret_cast<const uint32_t*>(codes + r * C + c));
      }
      const float sc = __ldg(scale + (per_row ? r : 0));
      v0 = __fmul_rn(sc, (float)(int8_t)(word & 0xFF));
      v1 = __fmul_rn(sc, (float)(int8_t)((word >> 8) & 0xFF));
      v2 = __fmul_rn(sc, (float)(int8_t)((word >> 16) & 0xFF));
      v3 = __fmul_rn(sc, (float)(int8_t)(word >> 24));
    }
    tile[i][4 * cw + 0] = v0;
    tile[i][4 * cw + 1] = v1;
    tile[i][4 * cw + 2] = v2;
    tile[i][4 * cw + 3] = v3;
  }
  __syncthreads();
  const int64_t s0 = r0 / chunk, in_chunk = r0 - s0 * chunk;  // the tile's chunk and its first row inside it
  for (int i = ty; i < kTrTile; i += 8) {
    const int64_t c = c0 + i;
    if (c >= C) continue;
    float* row = out + (s0 * rows_out + c) * chunk + in_chunk;
#pragma unroll
    for (int j = 0; j < kTrRows / 32; ++j)
      if (r0 + 32 * j + tx < r_pad) row[32 * j + tx] = tile[32 * j + tx][i];
  }
}

// x [R, C] floats with row pitch ldx -> value(r, c) = x[r][c] in the layout above.  If colsum_partial
// is not null, the block also writes the sums of its 128 rows of each of its columns, added top
// to bottom, to colsum_partial[blockIdx.y * C + c] (the first stage of a fixed-order column sum).
__global__ void __launch_bounds__(256) transpose_f32_kernel(const float* __restrict__ x, int64_t ldx, int64_t R, int64_t C,
                                                            float* __restrict__ out, int64_t r_pad, int64_t chunk, int64_t rows_out,
                                                            float* __restrict__ colsum_partial) {
  __shared__ float tile[kTrRows][kTrTile + 1];
  const int64_t r0 = (int64_t)blockIdx.y * kTrRows, c0 = (int64_t)blockIdx.x * kTrTile;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll 4
  for (int i = ty; i < kTrRows; i += 8) {
    const int64_t r = r0 + i, c = c0 + tx;
    tile[i][tx] = (r < R && c < C) ? __ldg(x + r * ldx + c) : 0.0f;
  }
  __syncthreads();
  const int64_t s0 = r0 / chunk, in_chunk = r0 - s0 * chunk;
  for (int i = ty; i < kTrTile; i += 8) {
    const int64_t c = c0 + i;
    if (c >= C) continue;
    float* row = out + (s0 * rows_out + c) * chunk + in_chunk;
#pragma unroll
    for (int j = 0; j < kTrRows / 32; ++j)
      if (r0 + 32 * j + tx < r_pad) row[32 * j + tx] = tile[32 * j + tx][i];
  }
  if (colsum_partial != nullptr && ty == 0 && c0 + tx < C) {
    float t = 0.0f;
    for (int i = 0; i < kTrRows; ++i) t = __fadd_rn(t, tile[i][tx]);  // rows beyond R hold zeros
    colsum_partial[(int64_t)blockIdx.y * C + c0 + tx] = t;
  }
}

// out[n][k] (row pitch ldo) = sum over batches s of partial[(s * rows_p + n) * K + k], in order.
__global__ void __launch_bounds__(256) sum_batches_kernel(const float* __restrict__ partial, int64_t batches, int64_t rows_p, int64_t N,
                                                          int64_t K, float* __restrict__ out, int64_t ldo) {
  const int64_t k4 = K >> 2, total = N * k4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t n = i / k4, c = i - n * k4;
    float4 t = __ldg(reinterpret_cast<const float4*>(partial + n * K) + c);
    for (int64_t s = 1; s < batches; ++s) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(partial + (s * rows_p + n) * K) + c);
      t.x = __fadd_rn(t.x, v.x);
      t.y = __fadd_rn(t.y, v.y);
      t.z = __fadd_rn(t.z, v.z);
      t.w = __fadd_rn(t.w, v.w);
    }
    reinterpret_cast<float4*>(out + n * ldo)[c] = t;
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
  // 32 columns per block; thread (tx, ty) adds the chunks j = ty, ty + 8, ... of column tx in order,
  // then the eight sums of a column are added in order: a fixed grouping, the same bits on every run
  __shared__ float acc[8][kTrTile];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t c = (int64_t)blockIdx.x * kTrTile + tx;
  float t = 0.0f;
  if (c < C)
    for (int64_t j = ty; j < chunks; j += 8) t = __fadd_rn(t, __ldg(partial + j * C + c));
  acc[ty][tx] = t;
  __syncthreads();
  if (ty == 0 && c < C) {
    float u = acc[0][tx];
#pragma unroll
    for (int i = 1; i < 8; ++i) u = __fadd_rn(u, acc[i][tx]);
    out[c] = u;
  }
}

__global__ void __launch_bounds__(256) fill_f32_kernel(float* __restrict__ p, int64_t n, float v) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

// r_pad: rows of the input covered, zeros beyond R (batches * chunk, or the padded pitch for one chunk).
static int launch_transpose_scale_codes(const void* codes, bool packed, const float* scale, bool per_row, int64_t R, int64_t C, float* out,
                                        int64_t r_pad, int64_t chunk, int64_t rows_out, cudaStream_t st) {
  const dim3 grid((unsigned)ceil_div(C, kTrTile), (unsigned)ceil_div(r_pad, kTrRows));
  transpose_scale_codes_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const uint8_t*>(codes), packed, scale, per_row, R, C, out, r_pad,
                                                     chunk, rows_out);
  return AQT_LAUNCH_STATUS();
}
// colsum_partial / colsum_out: null, or the column sums of x are produced on the way
// (colsum_partial holds transpose_row_blocks(r_pad) * C floats).
static int64_t transpose_row_blocks(int64_t r_pad) { return ceil_div(r_pad, kTrRows); }
static int launch_colsum_stage2(const float* partial, int64_t chunks, int64_t C, float* out, cudaStream_t st);
static int launch_transpose_f32(const float* x, int64_t ldx, int64_t R, int64_t C, float* out, int64_t r_pad, int64_t chunk,
                                int64_t rows_out, float* colsum_partial, float* colsum_out, cudaStream_t st) {
  const dim3 grid((unsigned)ceil_div(C, kTrTile), (unsigned)transpose_row_blocks(r_pad));
  transpose_f32_kernel<<<grid, 256, 0, st>>>(x, ldx, R, C, out, r_pad, chunk, rows_out, colsum_partial);
  int rc = AQT_LAUNCH_STATUS();
  if (rc != AQT_OK || colsum_partial == nullptr) return rc;
  return launch_colsum_stage2(colsum_partial, transpose_row_blocks(r_pad), C, colsum_out, st);
}
static int launch_sum_batches(const float* partial, int64_t batches, int64_t rows_p, int64_t N, int64_t K, float* out, int64_t ldo,
                              cudaStream_t st) {
  const int64_t want = ceil_div(N * K / 4, 256);
  sum_batches_kernel<<<(unsigned)(want < 1 ? 1 : (want > 148 * 16 ? 148 * 16 : want)), 256, 0, st>>>(partial, batches, rows_p, N, K, out, ldo);
  return AQT_LAUNCH_STATUS();
}
static int64_t colsum_chunks(int64_t R) { return ceil_div(R, kColsumChunk); }
static int launch_colsum(const float* x, int64_t ldx, int64_t R, int64_t C, float* partial, float* out, cudaStream_t st) {
  const int64_t chunks = colsum_chunks(R);
  colsum_stage1_kernel<<<dim3((unsigned)ceil_div(C, kTrTile), (unsigned)chunks), 256, 0, st>>>(x, ldx, R, C, partial);
  int rc = AQT_LAUNCH_STATUS();
  if (rc != AQT_OK) return rc;
  colsum_stage2_kernel<<<(unsigned)ceil_div(C, kTrTile), 256, 0, st>>>(partial, chunks, C, out);
  return AQT_LAUNCH_STATUS();
}
static int launch_colsum_stage2(const float* partial, int64_t chunks, int64_t C, float* out, cudaStream_t st) {
  colsum_stage2_kernel<<<(unsigned)ceil_div(C, kTrTile), 256, 0, st>>>(partial, chunks, C, out);
  return AQT_LAUNCH_STATUS();
}
static int launch_fill_f32(float* p, int64_t n, float v, cudaStream_t st) {
  fill_f32_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(p, n, v);
  return AQT_LAUNCH_STATUS();
}

}  // namespace aqt
