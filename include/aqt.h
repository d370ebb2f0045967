/*
 * aqt.h -- C ABI of the quantized linear layer (native integer quantization, arXiv 2203.15952).
 *
 * The layer: dynamic abs-max symmetric quantization of activations to int8 / int4 codes plus
 * scales (Fig. 2, Section 2.2), pre-quantized per-output-channel int4 / int8 weights, an integer
 * matmul with int32 accumulation (Section 1: native integer operations), and de-quantization by
 * multiplying with the scales (Section 2.2) fused with bias, activation and residual.
 *
 * Conventions
 *  - Every function returns an int status: AQT_OK or a negative AQT_ERR_* code.  Nothing throws.
 *  - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.  The
 *    library allocates no device memory; scratch space is passed in as `workspace`.
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default
 *    stream) of the current device and is not synchronised.  Argument errors are reported
 *    synchronously by the return value and nothing is enqueued; device-side failures (a bounded
 *    wait that ran out) are recorded in a device status word read by aqt_device_status().
 *  - Outputs must not alias inputs.  Inputs must be finite (NaN / Inf: codes unspecified).
 *  - Matrices are row-major.  x is [M, K]; weights are handed over as W^T = [N, K] with K
 *    contiguous (row n = output channel n), so y = x . W with W = [K, N].
 *  - 4-bit codes are two's-complement nibbles, two per byte along K: even k in the low nibble,
 *    odd k in the high nibble.  The paper states only the resulting model sizes (Tables 1, 2);
 *    this layout is the library's.
 *  - Built for sm_100a only.  A call on another device returns AQT_ERR_UNSUPPORTED.
 */
#ifndef AQT_H_
#define AQT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AQT_VERSION 201

/* status codes */
#define AQT_OK 0
#define AQT_ERR_BADARG (-1)      /* null pointer, negative size, unknown enum value, odd K for int4 */
#define AQT_ERR_ALIGN (-2)       /* a base pointer or row pitch violates the stated alignment       */
#define AQT_ERR_UNSUPPORTED (-3) /* device is not sm_100, or a size is beyond the stated limits      */
#define AQT_ERR_WORKSPACE (-4)   /* workspace missing or smaller than aqt_workspace_bytes()          */
#define AQT_ERR_CUDA (-5)        /* a CUDA runtime / driver call failed                             */
#define AQT_ERR_TIMEOUT (-6)     /* a bounded device-side wait ran out (reported by aqt_device_status) */

/* which axis aqt_quantize reduces over (Fig. 2: reduce_max(abs(input), axis, keepdims=True)) */
#define AQT_AXIS_ROW 0    /* reduce over columns: one scale per row       -> scale_out[rows] */
#define AQT_AXIS_COL 1    /* reduce over rows: one scale per column       -> scale_out[cols] */
#define AQT_AXIS_TENSOR 2 /* reduce over all elements: one scale          -> scale_out[1]    */

/* rounding of scaled values to codes */
#define AQT_ROUND_HALF_UP_FLOOR 0 /* floor(v + 0.5), the sum rounded in binary32 (Fig. 2)  */
#define AQT_ROUND_NEAREST_EVEN 1  /* IEEE 754 round-to-nearest, ties to even               */

/* granularity of the activation scale handed to the matmul */
#define AQT_SCALE_ROW 0    /* s_x[M], one per row (reduced over K) */
#define AQT_SCALE_TENSOR 1 /* s_x[1]                               */

/* epilogue activation (not part of the paper; Conformer module definitions) */
#define AQT_ACT_NONE 0
#define AQT_ACT_SWISH 1     /* a = z * sigmoid(z)                                              */
#define AQT_ACT_GLU 2       /* a[j] = z[j] * sigmoid(z[j + N/2]), j < N/2; output has N/2 columns */
#define AQT_ACT_GLU_SWISH 3 /* Swish applied to the GLU output                                  */

/* operand widths of the matmul entry points (bits_a, bits_w).  Fig. 2 keeps 4-bit codes in an
 * 8-bit container; the packed form is this library's storage layout. */
#define AQT_BITS_4_UNPACKED 48 /* 4-bit codes, one per int8 container: what aqt_quantize(bits 4, pack 0) and
                                  aqt_unpack_int4 produce.  Same layout as 8-bit codes; the smaller range lets the
                                  epilogue convert accumulators on the plain ALUs up to a deeper K. */

#define AQT_STATIC_WEIGHTS 0x100 /* may be OR-ed into bits_w of the matmul entry points: the weight codes, their scales and
                                    the bias were complete before the work that precedes this call on the stream was enqueued
                                    (weights of a trained model, as opposed to weights re-quantized by the preceding call).
                                    The kernels then fetch their weights while the preceding kernel is still draining;
                                    everything else they touch still waits for it. */

/* operations for aqt_workspace_bytes */
#define AQT_OP_QMATMUL 1
#define AQT_OP_LINEAR_FWD 2
#define AQT_OP_QMATMUL_REQUANT 3
#define AQT_OP_LINEAR_WEIGHT_ONLY 4    /* precision AQT_FLOAT_TF32   */
#define AQT_OP_LINEAR_WEIGHT_ONLY_X2 5 /* precision AQT_FLOAT_TF32X2 */
#define AQT_OP_LINEAR_BWD 6
#define AQT_OP_FFN_FWD 7 /* N = feed-forward width, K = model width, bits_w for both layers */

/* how float activations enter the tensor-core float matmul of the weight-only layer */
#define AQT_FLOAT_TF32 0   /* one term: the upper ten fraction bits of each activation            */
#define AQT_FLOAT_TF32X2 1 /* two terms x = hi + lo: about twenty-one significant bits, twice the work */

int aqt_version(void);
const char* aqt_status_string(int status);

/*
 * aqt_quantize -- Fig. 2, quantize(input, axis), and its int4 form (Section 2.2: divide the
 * abs-max by 7 instead of 127).
 *   amax  = max |x| over the reduced axis;  scale = amax / qmax, qmax = 127 (bits 8) or 7 (bits 4)
 *   v     = x / scale (0 where scale == 0, "divide_no_nan"), IEEE binary32 division
 *   code  = floor(v + 0.5) or nearest-even(v) per `rounding`, clipped to +-qmax as a guard
 * x         [rows, cols] fp32, row pitch ld elements (ld >= cols).
 * q_out     pack == 0: int8 [rows, cols] dense (both bit widths use an int8 container, as the
 *           figure's cast does).  pack == 1 (bits == 4 only, cols even): uint8 [rows, cols/2].
 * scale_out fp32, extent given by `axis` (see AQT_AXIS_*).  For AQT_AXIS_COL and
 *           AQT_AXIS_TENSOR it also serves as the abs-max accumulator while the call runs.
 * Alignment: none required; 16-byte aligned x with ld % 4 == 0 and cols % 4 == 0 takes the
 * vectorised path.  rows or cols == 0 is a no-op.
 */
int aqt_quantize(const float* x, int64_t rows, int64_t cols, int64_t ld, int bits, int axis, int rounding,
                 int pack, void* q_out, float* scale_out, void* stream);

/*
 * aqt_pack_int4 / aqt_unpack_int4 -- 4-bit storage of codes (the paper reports only model sizes,
 * Tables 1 and 2; nibble order as stated at the top).  q is int8 [rows, cols] with values in
 * [-8, 7]; packed is uint8 [rows, cols/2]; cols must be even (AQT_ERR_BADARG otherwise).
 * Unpacking sign-extends each nibble, which is exact.
 */
int aqt_pack_int4(const int8_t* q, int64_t rows, int64_t cols, uint8_t* packed, void* stream);
int aqt_unpack_int4(const uint8_t* packed, int64_t rows, int64_t cols, int8_t* q, void* stream);

/*
 * aqt_qmatmul -- integer matmul on codes with the de-quantizing epilogue (Section 1: native
 * integer matmul; Section 2.2: de-quantize by multiplying with the scales):
 *   acc[m][n] = sum_k xq[m][k] * wq[n][k]                      exact, int32
 *   z[m][n]   = fma(float(acc) * s_x[m or 0], s_w[n], bias[n]) binary32, bias = 0 if NULL
 *   a         = act(z)                                         see AQT_ACT_*
 *   y         = residual ? fma(residual_scale, a, residual) : a
 * xq        bits_a == 8 or AQT_BITS_4_UNPACKED: int8 [M, K];  bits_a == 4: uint8 [M, K/2] packed.
 * s_x       fp32 [M] (AQT_SCALE_ROW) or [1] (AQT_SCALE_TENSOR).
 * wq        W^T codes: bits_w == 8 or AQT_BITS_4_UNPACKED: int8 [N, K];  bits_w == 4: uint8 [N, K/2] packed.
 *           (Weights with K > 512 that are used call after call are best unpacked once with
 *           aqt_unpack_int4 and handed over as AQT_BITS_4_UNPACKED: the packed form is otherwise
 *           sign-extended into the workspace on every call.)
 * s_w       fp32 [N];  bias fp32 [N] or NULL.
 * residual  fp32 [M, N_out] with row pitch ldr, or NULL.  N_out = N, or N/2 for the GLU forms.
 * y         fp32 [M, N_out], row pitch ldy.
 * acc_debug NULL, or int32 [M, N] dense: receives the raw accumulators (for parity checks).
 * workspace at least aqt_workspace_bytes(AQT_OP_QMATMUL, ...) bytes, 256-byte aligned; holds the
 *           sign-extended copy of each 4-bit operand.  May be NULL when both operands are 8-bit.
 * Limits: K % 16 == 0; N % 4 == 0 (N % 8 == 0 for GLU); ldy % 4 == 0, ldr % 4 == 0; xq, wq, y,
 * residual, s_w, bias 16-byte aligned; M, N, K < 2^31 and M*N < 2^40.  K <= 133 000 keeps every
 * accumulator inside int32.  M == 0 or N == 0 is a no-op.
 */
int aqt_qmatmul(const void* xq, const float* s_x, int s_x_kind, const void* wq, const float* s_w,
                const float* bias, const float* residual, int64_t ldr, float residual_scale, int64_t M,
                int64_t N, int64_t K, int bits_a, int bits_w, int act, float* y, int64_t ldy,
                int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream);

/*
 * aqt_plan_qmatmul -- names the kernel configuration aqt_qmatmul (and every entry point that runs
 * the same matmul) would launch for a shape: "small_m", "ws128e16", "pair256s6e4", ...  Host-only:
 * sm_count_or_0 > 0 plans for a device with that many multiprocessors, 0 for the current device
 * (148 if there is none).  float_kind != 0 plans the float matmul of aqt_linear_fwd_weight_only /
 * aqt_linear_bwd with K in elements.  (No counterpart in the paper: the choice of tile shapes is
 * this library's.)  name_out receives a NUL-terminated string of at most name_bytes bytes.
 */
int aqt_plan_qmatmul(int64_t M, int64_t N, int64_t K, int bits_a, int bits_w, int act, int float_kind,
                     int sm_count_or_0, char* name_out, size_t name_bytes);

/*
 * aqt_qmatmul_with_plan -- aqt_qmatmul run with the kernel configuration named `plan` (a host
 * string as returned by aqt_plan_qmatmul, except "small_m") instead of the one the library would
 * choose.  For tests and tuning: results are identical whatever the plan (the integer sums are
 * exact and the epilogue arithmetic is the same).  AQT_ERR_BADARG for an unknown name,
 * AQT_ERR_UNSUPPORTED if that configuration cannot run the shape.  Other arguments as aqt_qmatmul.
 */
int aqt_qmatmul_with_plan(const char* plan, const void* xq, const float* s_x, int s_x_kind, const void* wq,
                          const float* s_w, const float* bias, const float* residual, int64_t ldr,
                          float residual_scale, int64_t M, int64_t N, int64_t K, int bits_a, int bits_w, int act,
                          float* y, int64_t ldy, int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                          void* stream);

/*
 * aqt_qmatmul_requant -- aqt_qmatmul whose output rows are quantized for the next layer inside
 * the same kernel (Section 2.2: every quantized layer quantizes its input dynamically, so the
 * tensor between two such layers is only ever consumed as codes and row scales; Fig. 2 is
 * applied to the output rows before they leave the SM, and the fp32 tensor is not written
 * unless the caller asks for it):
 *   u            = what aqt_qmatmul would write to y (same arguments, same arithmetic)
 *   q_out, s_out = aqt_quantize(u, axis = AQT_AXIS_ROW, bits_out, rounding, pack_out)
 * q_out     bits_out == 8 or pack_out == 0: int8 [M, N_out] dense;  pack_out == 1 (bits_out == 4
 *           only): uint8 [M, N_out/2] packed.
 * s_out     fp32 [M].
 * y         NULL, or fp32 [M, N_out] with row pitch ldy: also receives u (a residual stream, or
 *           a parity check).  residual != NULL requires y != NULL.
 * workspace at least aqt_workspace_bytes(AQT_OP_QMATMUL_REQUANT, ...) bytes, 256-byte aligned:
 *           what aqt_qmatmul needs plus the area through which CTAs exchange row maxima.
 * Limits: those of aqt_qmatmul, and N_out % 16 == 0 (N_out % 32 == 0 if pack_out).  One kernel
 * does both steps for: K <= 512 with act NONE or SWISH; the GLU forms when only int8 codes and
 * scales are asked for (y == NULL, pack_out == 0); 512 < K <= 1024 when y == NULL; and K >= 2048
 * with act NONE or SWISH, M > 128, N <= 2048 and pack_out == 0 (with or without y).  The CTAs of
 * such a kernel wait on one another (row maxima cross CTAs), with the same bounded waits as
 * everything else, so it runs on at most one CTA per SM and reports AQT_ERR_TIMEOUT through the
 * device status word if other work keeps SMs from it for seconds.  Other calls run the two
 * steps one after the other through y and return AQT_ERR_UNSUPPORTED if y is NULL.
 */
int aqt_qmatmul_requant(const void* xq, const float* s_x, int s_x_kind, const void* wq, const float* s_w,
                        const float* bias, const float* residual, int64_t ldr, float residual_scale, int64_t M,
                        int64_t N, int64_t K, int bits_a, int bits_w, int act, int bits_out, int rounding,
                        int pack_out, void* q_out, float* s_out, float* y, int64_t ldy, void* workspace,
                        size_t workspace_bytes, void* stream);

/*
 * aqt_linear_fwd -- the whole layer for fp32 activations: aqt_quantize(x, axis = K) with a
 * per-row or per-tensor dynamic scale, then aqt_qmatmul (same arguments and limits).
 * x         fp32 [M, K], row pitch ldx.
 * workspace at least aqt_workspace_bytes(AQT_OP_LINEAR_FWD, ...) bytes, 256-byte aligned; holds
 *           the activation codes and scales between the two steps and what aqt_qmatmul needs.
 */
int aqt_linear_fwd(const float* x, int64_t ldx, const void* wq, const float* s_w, const float* bias,
                   const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K,
                   int bits_a, int bits_w, int a_scale_kind, int rounding, int act, float* y, int64_t ldy,
                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * aqt_linear_fwd_host -- aqt_linear_fwd for callers whose activations live in HOST memory
 * (Section 2.2's layer, unchanged; only where x and y live differs).
 * x         fp32 [M, K] dense: a host pointer if x_on_host != 0, else a device pointer.
 * y         fp32 [M, N_out] dense: a host pointer if y_on_host != 0, else a device pointer.
 *           Pinned host memory makes the copies asynchronous.  Weights, scales and bias are
 *           device pointers as everywhere else.  No residual input.
 * workspace device memory, at least aqt_workspace_bytes(AQT_OP_LINEAR_FWD, ...) rounded up to
 *           256, plus 4*M*K rounded up to 256 if x_on_host, plus 4*M*N_out if y_on_host: the
 *           device copies of x and y are placed behind the layer's own scratch, in that order.
 * The call enqueues the host-to-device copy, the layer and the device-to-host copy on `stream`
 * and returns without synchronising.  Chaining two calls (host -> device, device -> host) runs a
 * two-layer block with only its input and output crossing the bus.
 */
int aqt_linear_fwd_host(const float* x, int x_on_host, const void* wq, const float* s_w, const float* bias,
                        int64_t M, int64_t N, int64_t K, int bits_a, int bits_w, int a_scale_kind, int rounding,
                        int act, float* y, int y_on_host, void* workspace, size_t workspace_bytes, void* stream);

/*
 * aqt_ffn_fwd -- a feed-forward pair of quantized layers, y = W2 . act(W1 . x), each layer the
 * quantized linear layer of this library (Fig. 2 on its input rows, integer matmul, Section 2.2
 * de-quantization): aqt_quantize(x) -> aqt_qmatmul_requant (the hidden tensor u = act(W1 . x)
 * leaves the first matmul as codes and row scales and is never written as fp32) -> aqt_qmatmul.
 * x, y      fp32 [M, d] dense; host pointers if x_on_host / y_on_host != 0 (pinned memory makes
 *           the copies asynchronous), else device pointers.  The copies are enqueued on `stream`.
 * w1q       W1^T codes [ff, d], s_w1 [ff], bias1 [ff] or NULL, bits_w1 as for aqt_qmatmul.
 * w2q       W2^T codes [d, ff], s_w2 [d], bias2 [d] or NULL, bits_w2.
 * bits_a    4 or 8: width both layers' activations are quantized to (per-row dynamic scales).
 * act       AQT_ACT_NONE or AQT_ACT_SWISH between the layers.
 * workspace at least aqt_workspace_bytes(AQT_OP_FFN_FWD, M, ff, d, bits_a, bits_w) bytes (sized for
 *           host x and y and for one weight width: pass the wider of bits_w1 / bits_w2), 256-byte aligned.
 * Limits: d <= 1024 and the limits of aqt_qmatmul_requant's fused form (AQT_ERR_UNSUPPORTED otherwise).
 */
int aqt_ffn_fwd(const float* x, int x_on_host, const void* w1q, const float* s_w1, const float* bias1, int bits_w1,
                const void* w2q, const float* s_w2, const float* bias2, int bits_w2, int64_t M, int64_t d, int64_t ff,
                int bits_a, int rounding, int act, float* y, int y_on_host, void* workspace, size_t workspace_bytes,
                void* stream);

/*
 * aqt_linear_fwd_weight_only -- the layer of the weight-only configurations of Section 4.1 (I8W
 * and I4W: 8- or 4-bit weight codes against unquantized binary32 activations; the section notes
 * that the codes have to be turned back into floats when the layer runs).  Activations are not quantized; the stored
 * codes are converted to float and de-quantized by their channel scale (Section 2.2):
 *   z[m][n] = s_w[n] * sum_k x[m][k] * float(wq[n][k]) + bias[n]
 *   a = act(z);  y = residual ? fma(residual_scale, a, residual) : a
 * Arithmetic: a float matmul on the tensor cores.  The weight codes are exact as floats; each
 * activation enters its product with sign, exponent and the upper ten fraction bits of its
 * binary32 value (the tf32 operand format; whether the dropped bits are truncated or rounded is
 * the hardware's), products are exact and are summed into binary32 accumulators.  The result is
 * therefore within 2^-10 * s_w[n] * sum_k |x[m][k] * wq[n][k]| (plus binary32 summation error) of
 * the exact value of the formula, and equals it bit for bit when every x is a tf32 value and no
 * partial sum needs more than 24 bits.
 * precision AQT_FLOAT_TF32: as just described.  AQT_FLOAT_TF32X2: every activation is split
 *           exactly into hi (its tf32 part) + lo, and one matmul over [hi | lo] against the
 *           weights repeated sums both terms: the operand error drops from 2^-10 to 2^-20 of
 *           the terms' magnitude for twice the tensor-core work and one more pass over x.
 * x         fp32 [M, K], row pitch ldx elements.
 * wq, s_w, bias, residual, ldr, residual_scale, act, y, ldy: as for aqt_qmatmul.
 * workspace at least aqt_workspace_bytes(AQT_OP_LINEAR_WEIGHT_ONLY or .._X2, M, N, K, 0, bits_w)
 *           bytes, 256-byte aligned: the weight codes as floats (4 * N * K bytes; X2: 8 * N * K
 *           and the split activations, 8 * M * K), rewritten every call.
 * Limits: K % 4 == 0, ldx % 4 == 0, N % 4 == 0 (N % 8 == 0 for GLU), ldy % 4 == 0, ldr % 4 == 0;
 * x, wq, y, residual, s_w, bias 16-byte aligned.  M == 0 or N == 0 is a no-op.
 */
int aqt_linear_fwd_weight_only(const float* x, int64_t ldx, const void* wq, const float* s_w, const float* bias,
                               const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K,
                               int bits_w, int precision, int act, float* y, int64_t ldy, void* workspace,
                               size_t workspace_bytes, void* stream);

/*
 * aqt_linear_bwd -- backward of the quantized linear layer with straight-through quantizers.
 * The paper states that scales carry no gradient (Fig. 2: stop_gradient(scale)) and that training
 * runs the same integer forward (Section 1); it does not print the backward products.  This is
 * the plain straight-through definition: with xhat = s_x * xq and what = s_w * wq the de-quantized
 * operands of the forward y = xhat . what^T + bias, quantizers passing gradients unchanged,
 *   dx[m][k] = sum_n dy[m][n] * s_w[n] * wq[n][k]
 *   dw[n][k] = sum_m dy[m][n] * s_x[m or 0] * xq[m][k]      (the [N, K] layout of the weight codes)
 *   dbias[n] = sum_m dy[m][n]
 * dy is the gradient with respect to the layer's pre-activation (for a layer with an activation
 * or a residual the caller applies those derivatives first).
 * Arithmetic: dx and dw are float matmuls on the tensor cores (tf32 operands: dy and the scaled
 * codes each enter with their upper ten fraction bits; binary32 accumulation), so each is within
 * (2^-9 + depth * 2^-24) of the sum of the absolute values of its terms, depth = N for dx, M for
 * dw.  dbias is summed in binary32 in a fixed order (the same bits on every run).
 * dy        fp32 [M, N], row pitch lddy.
 * xq, s_x, s_x_kind, bits_a   the forward's activation codes and scales (as handed to aqt_qmatmul);
 *           only read for dw.
 * wq, s_w, bits_w             the weight codes and scales; only read for dx.
 * dx        fp32 [M, K], row pitch lddx, or NULL.   dw  fp32 [N, K], row pitch lddw, or NULL.
 * dbias     fp32 [N] or NULL.
 * workspace at least aqt_workspace_bytes(AQT_OP_LINEAR_BWD, M, N, K, 0, 0) bytes, 256-byte
 *           aligned: the transposed, scaled operands (4 * (K * N + (N + K) * M) bytes and change)
 *           and, where the weight gradient's contraction is split over CTAs, the partial products.
 * Limits: K % 4 == 0, N % 4 == 0; lddy, lddx, lddw multiples of 4; dy, dx, dw, xq, wq 16-byte aligned;
 * M, N < 2^23, K < 2^28 (larger sizes return AQT_ERR_UNSUPPORTED before anything is enqueued).  M == 0 or N == 0 is a no-op.
 */
int aqt_linear_bwd(const float* dy, int64_t lddy, const void* xq, const float* s_x, int s_x_kind, int bits_a,
                   const void* wq, const float* s_w, int bits_w, int64_t M, int64_t N, int64_t K, float* dx,
                   int64_t lddx, float* dw, int64_t lddw, float* dbias, void* workspace, size_t workspace_bytes,
                   void* stream);

/*
 * aqt_qmatmul_w4_noalloc -- aqt_qmatmul for int8 activations and 4-bit weights that needs no
 * workspace from the caller.  (The paper has no counterpart; this is a packaging variant of the
 * call above.)
 *
 * Who it is for: callers that cannot obtain device scratch memory at all -- code running where
 * cudaMalloc is forbidden or unavailable (inside a stream capture, in a plugin whose host owns
 * every allocation, under a fixed memory budget with no allocator hook).  The sign-extended copy
 * of the weights, which aqt_qmatmul places in `workspace`, is placed here in an array that is
 * part of the library image itself: AQT_NOALLOC_MAX_WEIGHT_BYTES bytes of device memory that
 * every GPU holding the library keeps until the process exits.
 *
 * Arguments, layouts, limits and results are those of aqt_qmatmul with bits_a = 8, bits_w = 4,
 * acc_debug = NULL and no workspace.  Additional rules:
 *  - N * K must not exceed AQT_NOALLOC_MAX_WEIGHT_BYTES; larger weights return
 *    AQT_ERR_UNSUPPORTED and nothing is enqueued.
 *  - The first call on each device looks up the array's device address (one runtime query, no
 *    allocation) with that device current; make that first call outside any stream capture.
 *  - The call allocates nothing and calls no allocating routine.
 *  - All calls on a device share the one array, and it keeps the previous call's bytes.  Each
 *    call rewrites the N * K bytes it uses before reading them, so nothing needs clearing; but two
 *    calls that overlap on the GPU (different streams, no ordering between them) race on it and
 *    produce garbage.  Order them on one stream or with events.
 */
#define AQT_NOALLOC_MAX_WEIGHT_BYTES (4u << 20)
int aqt_qmatmul_w4_noalloc(const int8_t* xq, const float* s_x, int s_x_kind, const uint8_t* wq_packed,
                           const float* s_w, const float* bias, const float* residual, int64_t ldr,
                           float residual_scale, int64_t M, int64_t N, int64_t K, int act, float* y,
                           int64_t ldy, void* stream);

/* Scratch bytes needed by `op` (AQT_OP_*) at these sizes; 0 if none.  Host-only, no CUDA call. */
size_t aqt_workspace_bytes(int op, int64_t M, int64_t N, int64_t K, int bits_a, int bits_w);

/*
 * aqt_device_status -- synchronises `stream`, copies the device status word to *status_out (host
 * pointer) and clears it.  AQT_OK, or AQT_ERR_TIMEOUT if a kernel gave up on a bounded wait since
 * the last call (its output is then undefined).  Returns AQT_ERR_CUDA if the copy itself failed.
 */
int aqt_device_status(void* stream, int* status_out);

/*
 * aqt_selftest_bounded_wait -- exercises the failure path of the kernels' bounded waits without
 * hanging anything: one CTA waits, for at most limit_ns (1 .. 10^9), on a barrier that nothing
 * signals.  The wait gives up, the kernel returns normally, *gave_up_dev (device int) is set to 1
 * and the device status word to AQT_ERR_TIMEOUT, which the next aqt_device_status() reports and
 * clears.  (The paper has no counterpart: this is the library's own fault-reporting check.)
 */
int aqt_selftest_bounded_wait(uint64_t limit_ns, int* gave_up_dev, void* stream);

/*
 * aqt_selftest_sfu_rate -- a measurement aid: launches a kernel that does nothing but the two
 * special-function operations of the Swish / GLU epilogues (2^x and reciprocal) in independent
 * chains on every SM, `iterations` (1 .. 2^20) rounds of 16 operations per thread.  *ops_out
 * (host) receives the number of operations the launch performs; the caller times the launch
 * (CUDA events) to get the device's special-function rate, the ceiling the activation epilogues
 * are measured against.  sink_dev: one device float, never written in practice.  (The paper has
 * no counterpart.)
 */
int aqt_selftest_sfu_rate(int iterations, float* sink_dev, int64_t* ops_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AQT_H_ */
