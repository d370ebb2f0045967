/*
 * CPU oracle for the quantized linear layer of "4-bit Conformer with Native Quantization Aware
 * Training for Speech Recognition" (arXiv 2203.15952).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the layer computes.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may call it; the
 * library's product path never does.  It shares no code, header, table or helper with the CUDA
 * implementation.
 *
 * What is written out here, in the paper's order:
 *   Fig. 2 / Section 2.2 : the dynamic symmetric quantizer.  The largest magnitude along the
 *                          reduced axis, divided by the largest code (127 at 8 bits, 7 at 4 bits),
 *                          is the scale; every element is divided by its scale (zero where the
 *                          scale is zero), rounded half-up by a floor, and kept in an 8-bit
 *                          container.
 *   Section 2.2          : the scheme is symmetric (no zero point), and a code times its scale
 *                          gives the value back.
 *   Section 1            : the matmul runs natively on the integer codes; emulating it in
 *                          binary32 stops being exact once sums outgrow the significand.
 * Readings taken where the paper is silent are stated beside each function.
 *
 * Parity status of each function (what pins it, independent of this file) is listed in
 * oracle/README.md; functions that no published value or identity pins say "parity unpinned"
 * there.  Nothing in the paper prints a worked numeric example, so every pin is an invariant,
 * a closed form, a brute-force enumeration or a special case that reduces to a textbook result.
 *
 * Build: gcc -O2 -std=c11 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 * Float arithmetic is IEEE binary32 exactly as written (SSE scalar ops, no contraction, no
 * flush-to-zero).  OpenMP only distributes independent rows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_AXIS_ROW 0    /* reduce over columns: one scale per row            */
#define ORC_AXIS_COL 1    /* reduce over rows: one scale per column            */
#define ORC_AXIS_TENSOR 2 /* reduce over everything: one scale                 */

#define ORC_ROUND_HALF_UP_FLOOR 0 /* floor(v + 0.5), Fig. 2                    */
#define ORC_ROUND_NEAREST_EVEN 1  /* IEEE round-to-nearest-even                */

#define ORC_ACT_NONE 0
#define ORC_ACT_SWISH 1
#define ORC_ACT_GLU 2
#define ORC_ACT_GLU_SWISH 3

#define ORC_SCALE_ROW 0
#define ORC_SCALE_TENSOR 1

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Largest code of a b-bit symmetric quantizer, 2^(b-1) - 1: the divisors 127 and 7 of Section 2.2. */
static int qmax_of(int bits) { return bits == 8 ? 127 : (bits == 4 ? 7 : -1); }

/* One element of Fig. 2 once its scale is known.
 * The quotient is defined as 0 where the scale is 0 (the figure uses a division that returns 0
 * instead of NaN or Inf there).
 * Rounding: the figure adds one half and takes the floor, the sum being a binary32 value; the
 * alternative is IEEE nearest-even, which the workload definitions ask for.  Both are kept.
 * The final clip is a guard only: with abs-max scaling |v| <= qmax up to one rounding, so the
 * clip acts only when the scale is subnormal and the quotient loses precision.  The method
 * itself has no clipping range to learn or apply (Section 1). */
static int8_t quantize_one(float x, float scale, int qmax, int rounding) {
  float v = (scale == 0.0f) ? 0.0f : x / scale;
  float r;
  if (rounding == ORC_ROUND_HALF_UP_FLOOR) {
    volatile float t = v + 0.5f; /* binary32 sum, then floor */
    r = floorf(t);
  } else {
    r = nearbyintf(v); /* default rounding mode: nearest, ties to even */
  }
  if (r > (float)qmax) r = (float)qmax;
  if (r < -(float)qmax) r = -(float)qmax;
  return (int8_t)r;
}

/* The quantizer of Fig. 2.  x is [rows, cols], row pitch ld (elements).
 * axis names the axis that is REDUCED (the figure's maximum keeps that axis with extent 1), so
 * there is one scale per slice across it: ORC_AXIS_ROW -> scale[rows], ORC_AXIS_COL ->
 * scale[cols], ORC_AXIS_TENSOR -> scale[1].  q is [rows, cols] dense in an 8-bit container for
 * both bit widths, as in the figure.  Returns 0, or -1 on a bad argument. */
int orc_quantize(const float* x, int64_t rows, int64_t cols, int64_t ld, int bits, int axis,
                 int rounding, int8_t* q, float* scale) {
  const int qmax = qmax_of(bits);
  if (qmax < 0 || rows < 0 || cols < 0 || ld < cols) return -1;
  if (rounding != ORC_ROUND_HALF_UP_FLOOR && rounding != ORC_ROUND_NEAREST_EVEN) return -1;
  if (axis == ORC_AXIS_ROW) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
      float amax = 0.0f;
      for (int64_t j = 0; j < cols; ++j) {
        float a = fabsf(x[i * ld + j]);
        if (a > amax) amax = a;
      }
      float s = amax / (float)qmax;
      scale[i] = s;
      for (int64_t j = 0; j < cols; ++j) q[i * cols + j] = quantize_one(x[i * ld + j], s, qmax, rounding);
    }
  } else if (axis == ORC_AXIS_COL) {
    for (int64_t j = 0; j < cols; ++j) {
      float amax = 0.0f;
      for (int64_t i = 0; i < rows; ++i) {
        float a = fabsf(x[i * ld + j]);
        if (a > amax) amax = a;
      }
      scale[j] = amax / (float)qmax;
    }
    for (int64_t i = 0; i < rows; ++i)
      for (int64_t j = 0; j < cols; ++j) q[i * cols + j] = quantize_one(x[i * ld + j], scale[j], qmax, rounding);
  } else if (axis == ORC_AXIS_TENSOR) {
    float amax = 0.0f;
    for (int64_t i = 0; i < rows; ++i)
      for (int64_t j = 0; j < cols; ++j) {
        float a = fabsf(x[i * ld + j]);
        if (a > amax) amax = a;
      }
    float s = amax / (float)qmax;
    scale[0] = s;
    for (int64_t i = 0; i < rows; ++i)
      for (int64_t j = 0; j < cols; ++j) q[i * cols + j] = quantize_one(x[i * ld + j], s, qmax, rounding);
  } else {
    return -1;
  }
  return 0;
}

/* Section 2.2: de-quantization is one multiply of each code by its scale.
 * `axis` selects which scale element applies (row i, column j, or the single one). */
int orc_dequantize(const int8_t* q, int64_t rows, int64_t cols, const float* scale, int axis, float* x) {
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      float s = axis == ORC_AXIS_ROW ? scale[i] : (axis == ORC_AXIS_COL ? scale[j] : scale[0]);
      x[i * cols + j] = (float)q[i * cols + j] * s;
    }
  return 0;
}

/* 4-bit storage.  The paper gives only the resulting model sizes (Table 1, Table 2); the layout
 * is this library's: two's-complement nibbles, two per byte along the row, even column in the
 * low nibble, odd column in the high nibble.  cols must be even. */
int orc_pack_int4(const int8_t* q, int64_t rows, int64_t cols, uint8_t* packed) {
  if (cols % 2 != 0) return -1;
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols / 2; ++j) {
      uint8_t lo = (uint8_t)q[i * cols + 2 * j] & 0xF;
      uint8_t hi = (uint8_t)q[i * cols + 2 * j + 1] & 0xF;
      packed[i * (cols / 2) + j] = (uint8_t)(lo | (hi << 4));
    }
  return 0;
}

static int8_t sext4(uint8_t nib) { return (int8_t)((nib & 0x8) ? (int)nib - 16 : (int)nib); }

int orc_unpack_int4(const uint8_t* packed, int64_t rows, int64_t cols, int8_t* q) {
  if (cols % 2 != 0) return -1;
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols / 2; ++j) {
      uint8_t b = packed[i * (cols / 2) + j];
      q[i * cols + 2 * j] = sext4(b & 0xF);
      q[i * cols + 2 * j + 1] = sext4(b >> 4);
    }
  return 0;
}

/* Bytes a quantized [K, N] weight occupies: codes at `bits` per entry plus one fp32 scale per
 * output channel.  bits = 32 means an unquantized fp32 weight (no scales). */
int64_t orc_weight_bytes(int64_t K, int64_t N, int bits) {
  if (bits == 32) return 4 * K * N;
  return (K * N * bits + 7) / 8 + 4 * N;
}

/* The integer matmul on codes (Section 1: quantized matrix products run as native integer
 * operations).  xq is [M, K]; wq holds W^T as [N, K] (row n is
 * output channel n).  acc[m][n] = sum_k xq[m][k] * wq[n][k] in 64-bit integers; integer sums do
 * not depend on the order of summation.  Returns how many results fall outside int32 (0 for
 * every K <= 133 000 at 8 bits). */
int64_t orc_int_matmul(const int8_t* xq, const int8_t* wq, int64_t M, int64_t N, int64_t K, int64_t* acc) {
  int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += (int64_t)xq[m * K + k] * (int64_t)wq[n * K + k];
      acc[m * N + n] = s;
      if (s > INT32_MAX || s < INT32_MIN) ++overflow;
    }
  return overflow;
}

/* The integer matmul emulated in binary32, the alternative Section 1 argues against: the same
 * codes converted to binary32, multiplied and summed left to right in binary32.  Used only to
 * test the paper's remark that emulation and integer math agree while results fit the significand. */
int orc_emulated_matmul_f32(const int8_t* xq, const int8_t* wq, int64_t M, int64_t N, int64_t K, float* out) {
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      volatile float s = 0.0f;
      for (int64_t k = 0; k < K; ++k) {
        volatile float p = (float)xq[m * K + k] * (float)wq[n * K + k];
        s = s + p;
      }
      out[m * N + n] = s;
    }
  return 0;
}

static double sigmoid_d(double z) { return 1.0 / (1.0 + exp(-z)); }

/* De-quantizing epilogue in the binary32 operation order the layer is specified with:
 *   t = float(acc) * s_x          (int -> float conversion to nearest-even, one rounded multiply)
 *   z = fma(t, s_w[n], bias[n])   (one rounding; bias = 0 when absent)
 * Section 2.2 only says that de-quantization multiplies by the scale; the order of the two
 * multiplies and the fp32 bias are this library's definition.
 * Activations (not in the paper; Conformer module definitions): evaluated in double on the
 * binary32 pre-activation z and rounded once to binary32:
 *   SWISH      a = z * sigmoid(z)
 *   GLU        a[j] = z[j] * sigmoid(z[j + N/2]),  j < N/2   (first half values, second half gates)
 *   GLU_SWISH  g = GLU in double, a = g * sigmoid(g)
 * Residual (optional): out = fma(residual_scale, a, residual) in binary32.
 * y has N columns (NONE, SWISH) or N/2 columns (GLU, GLU_SWISH), row pitch ldy; residual has the
 * same shape with pitch ldr.  z_out (optional, [M, N]) receives the pre-activations. */
int orc_epilogue_f32(const int64_t* acc, const float* s_x, int s_x_kind, const float* s_w, const float* bias,
                     const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int act,
                     float* y, int64_t ldy, float* z_out) {
  const int glu = (act == ORC_ACT_GLU || act == ORC_ACT_GLU_SWISH);
  if (glu && (N % 2 != 0)) return -1;
  const int64_t n_out = glu ? N / 2 : N;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    float* z = (float*)malloc((size_t)N * sizeof(float));
    const float sx = s_x_kind == ORC_SCALE_ROW ? s_x[m] : s_x[0];
    for (int64_t n = 0; n < N; ++n) {
      volatile float t = (float)(int32_t)acc[m * N + n] * sx;
      z[n] = fmaf(t, s_w[n], bias ? bias[n] : 0.0f);
      if (z_out) z_out[m * N + n] = z[n];
    }
    for (int64_t j = 0; j < n_out; ++j) {
      float a;
      if (act == ORC_ACT_NONE) {
        a = z[j];
      } else if (act == ORC_ACT_SWISH) {
        a = (float)((double)z[j] * sigmoid_d((double)z[j]));
      } else {
        double g = (double)z[j] * sigmoid_d((double)z[j + n_out]);
        a = (act == ORC_ACT_GLU) ? (float)g : (float)(g * sigmoid_d(g));
      }
      if (residual) a = fmaf(residual_scale, a, residual[m * ldr + j]);
      y[m * ldy + j] = a;
    }
    free(z);
  }
  return 0;
}

/* The same epilogue with every operation in double and no intermediate rounding: the value the
 * binary32 epilogue approximates.  Output is double, dense [M, n_out]. */
int orc_epilogue_f64(const int64_t* acc, const float* s_x, int s_x_kind, const float* s_w, const float* bias,
                     const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int act,
                     double* y) {
  const int glu = (act == ORC_ACT_GLU || act == ORC_ACT_GLU_SWISH);
  if (glu && (N % 2 != 0)) return -1;
  const int64_t n_out = glu ? N / 2 : N;
  for (int64_t m = 0; m < M; ++m) {
    const double sx = s_x_kind == ORC_SCALE_ROW ? (double)s_x[m] : (double)s_x[0];
    for (int64_t j = 0; j < n_out; ++j) {
      double z = (double)acc[m * N + j] * sx * (double)s_w[j] + (bias ? (double)bias[j] : 0.0);
      double a = z;
      if (act == ORC_ACT_SWISH) a = z * sigmoid_d(z);
      if (glu) {
        double zg = (double)acc[m * N + j + n_out] * sx * (double)s_w[j + n_out] + (bias ? (double)bias[j + n_out] : 0.0);
        a = z * sigmoid_d(zg);
        if (act == ORC_ACT_GLU_SWISH) a = a * sigmoid_d(a);
      }
      if (residual) a = (double)residual[m * ldr + j] + (double)residual_scale * a;
      y[m * n_out + j] = a;
    }
  }
  return 0;
}

/* The whole layer for fp32 activations x [M, K] (pitch ldx) and already-quantized weights
 * (codes wq as W^T [N, K] in int8 containers, scales s_w [N]): dynamic activation quantization
 * (per row, or per tensor), integer matmul, epilogue.  Optional outputs: xq_out [M, K] codes,
 * sx_out scales, acc_out [M, N] accumulators as int64.  Returns 0, -1 on bad arguments, -2 if an
 * accumulator left the int32 range. */
int orc_linear_fwd(const float* x, int64_t ldx, const int8_t* wq, const float* s_w, const float* bias,
                   const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K,
                   int bits_a, int a_scale_kind, int rounding, int act, float* y, int64_t ldy, int8_t* xq_out,
                   float* sx_out, int64_t* acc_out) {
  int8_t* xq = xq_out ? xq_out : (int8_t*)malloc((size_t)(M * K) + 1);
  float* sx = sx_out ? sx_out : (float*)malloc((size_t)(M + 1) * sizeof(float));
  int64_t* acc = acc_out ? acc_out : (int64_t*)malloc((size_t)(M * N + 1) * sizeof(int64_t));
  int rc = orc_quantize(x, M, K, ldx, bits_a, a_scale_kind == ORC_SCALE_ROW ? ORC_AXIS_ROW : ORC_AXIS_TENSOR,
                        rounding, xq, sx);
  if (rc == 0 && orc_int_matmul(xq, wq, M, N, K, acc) != 0) rc = -2;
  if (rc == 0)
    rc = orc_epilogue_f32(acc, sx, a_scale_kind, s_w, bias, residual, ldr, residual_scale, M, N, act, y, ldy, NULL);
  if (!xq_out) free(xq);
  if (!sx_out) free(sx);
  if (!acc_out) free(acc);
  return rc;
}

/* The layer of the weight-only configurations of Section 4.1 (I8W and I4W: 8- or 4-bit weight
 * codes against unquantized binary32 activations, the codes being turned back into floats when
 * the layer runs).  Activations are not quantized; de-quantization multiplies the codes by their
 * channel scale (Section 2.2).  The plain definition, every operation in double:
 *   z[m][n] = s_w[n] * sum_k x[m][k] * wq[n][k] + bias[n]
 * (each product of a binary32 value and a code is exact in double; the sum is rounded only at the
 * 2^-53 level.)  Activation and residual as in orc_epilogue_f64.
 * y is double [M, n_out] dense.  Optional outputs, double [M, N] dense: z_out, the
 * pre-activations; mag_out, s_w[n] * sum_k |x[m][k] * wq[n][k]|, the magnitude against which a
 * float implementation's rounding is measured. */
int orc_linear_weight_only_f64(const float* x, int64_t ldx, const int8_t* wq, const float* s_w, const float* bias,
                               const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N,
                               int64_t K, int act, double* y, double* z_out, double* mag_out) {
  const int glu = (act == ORC_ACT_GLU || act == ORC_ACT_GLU_SWISH);
  if (M < 0 || N < 0 || K < 0 || ldx < K) return -1;
  if (glu && (N % 2 != 0)) return -1;
  const int64_t n_out = glu ? N / 2 : N;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    double* z = (double*)malloc((size_t)(N + 1) * sizeof(double));
    for (int64_t n = 0; n < N; ++n) {
      double sum = 0.0, mag = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        double p = (double)x[m * ldx + k] * (double)wq[n * K + k];
        sum += p;
        mag += fabs(p);
      }
      z[n] = (double)s_w[n] * sum + (bias ? (double)bias[n] : 0.0);
      if (z_out) z_out[m * N + n] = z[n];
      if (mag_out) mag_out[m * N + n] = fabs((double)s_w[n]) * mag;
    }
    for (int64_t j = 0; j < n_out; ++j) {
      double a = z[j];
      if (act == ORC_ACT_SWISH) a = z[j] * sigmoid_d(z[j]);
      if (glu) {
        a = z[j] * sigmoid_d(z[j + n_out]);
        if (act == ORC_ACT_GLU_SWISH) a = a * sigmoid_d(a);
      }
      if (residual) a = (double)residual[m * ldr + j] + (double)residual_scale * a;
      y[m * n_out + j] = a;
    }
    free(z);
  }
  return 0;
}

/* Backward of the quantized linear layer with straight-through quantizers.  The paper states only
 * that the scale carries no gradient (Fig. 2: stop_gradient(scale)) and that training runs the
 * same integer forward that serving uses (Section 1); it does not print the
 * backward products.  The plain straight-through definition is taken: the forward is
 *   y[m][n] = sum_k xhat[m][k] * what[n][k] + bias[n],  xhat = s_x * xq,  what = s_w * wq,
 * the quantizers pass gradients through unchanged (d xhat / d x = 1, d what / d w = 1), scales are
 * constants.  With dy = dL/dy (for an activation the caller supplies dL/dz), every sum in double:
 *   dx[m][k] = sum_n dy[m][n] * s_w[n] * wq[n][k]
 *   dw[n][k] = sum_m dy[m][n] * s_x[m] * xq[m][k]       (same [N, K] layout as the codes)
 *   db[n]    = sum_m dy[m][n]
 * Optional magnitude outputs (sums of the absolute values of the same terms) bound the rounding
 * of float implementations.  Any output pointer may be NULL.  dy has row pitch lddy. */
int orc_linear_bwd_f64(const float* dy, int64_t lddy, const int8_t* xq, const float* s_x, int s_x_kind,
                       const int8_t* wq, const float* s_w, int64_t M, int64_t N, int64_t K, double* dx,
                       double* dw, double* db, double* dx_mag, double* dw_mag, double* db_mag) {
  if (M < 0 || N < 0 || K < 0 || lddy < N) return -1;
  if (dx) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
      for (int64_t k = 0; k < K; ++k) {
        double s = 0.0, a = 0.0;
        for (int64_t n = 0; n < N; ++n) {
          double t = (double)dy[m * lddy + n] * (double)s_w[n] * (double)wq[n * K + k];
          s += t;
          a += fabs(t);
        }
        dx[m * K + k] = s;
        if (dx_mag) dx_mag[m * K + k] = a;
      }
  }
  if (dw) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
      for (int64_t k = 0; k < K; ++k) {
        double s = 0.0, a = 0.0;
        for (int64_t m = 0; m < M; ++m) {
          double sx = s_x_kind == ORC_SCALE_ROW ? (double)s_x[m] : (double)s_x[0];
          double t = (double)dy[m * lddy + n] * sx * (double)xq[m * K + k];
          s += t;
          a += fabs(t);
        }
        dw[n * K + k] = s;
        if (dw_mag) dw_mag[n * K + k] = a;
      }
  }
  if (db) {
    for (int64_t n = 0; n < N; ++n) {
      double s = 0.0, a = 0.0;
      for (int64_t m = 0; m < M; ++m) {
        s += (double)dy[m * lddy + n];
        a += fabs((double)dy[m * lddy + n]);
      }
      db[n] = s;
      if (db_mag) db_mag[n] = a;
    }
  }
  return 0;
}
