// C ABI of the quantized linear layer: argument validation and kernel launches.
// Single translation unit: the kernels live in the headers included below.
#include "aqt_common.cuh"
#include "backward.cuh"
#include "pack.cuh"
#include "qgemm_sm100.cuh"
#include "qgemm_requant_sm100.cuh"
#include "qgemv_small_m.cuh"
#include "quantize.cuh"

using namespace aqt;

namespace {

// The kernels use tcgen05 / TMEM and exist for compute capability 10.x only.  Asked of the
// current device on every call (the answer is cached per device ordinal).
int check_device() {
  DeviceInfo d;
  int rc = current_device_info(&d);
  if (rc != AQT_OK) return rc;
  return d.cc_major == 10 ? AQT_OK : AQT_ERR_UNSUPPORTED;
}

// Operand widths a matmul accepts: 8, 4 (nibble-packed) or 4-bit codes in int8 containers.
bool bits_ok(int b) { return b == 4 || b == 8 || b == AQT_BITS_4_UNPACKED; }
bool quant_bits_ok(int b) { return b == 4 || b == 8; }
bool is_packed(int b) { return b == 4; }
int code_bits(int b) { return b == 8 ? 8 : 4; }  // range of the codes, whatever the container
bool act_ok(int a) { return a >= AQT_ACT_NONE && a <= AQT_ACT_GLU_SWISH; }
bool is_glu(int a) { return a == AQT_ACT_GLU || a == AQT_ACT_GLU_SWISH; }

size_t ws_qmatmul(int64_t M, int64_t N, int64_t K, int bits_a, int bits_w) {
  size_t b = 0;
  if (is_packed(bits_a)) b += round_up((size_t)M * (size_t)K, 256);
  if (is_packed(bits_w)) b += round_up((size_t)N * (size_t)K, 256);
  return b;
}
size_t ws_linear(int64_t M, int64_t N, int64_t K, int bits_w) {
  return round_up((size_t)M * (size_t)K, 256) + round_up((size_t)M * 4, 256) + ws_qmatmul(0, N, K, 8, bits_w);
}

// one-term form: the weights as floats; two-term form: the weights twice and the split activations
size_t ws_weight_only(int64_t M, int64_t N, int64_t K, int precision) {
  if (precision == AQT_FLOAT_TF32X2) return round_up((size_t)N * (size_t)K * 8, 256) + round_up((size_t)M * (size_t)K * 8, 256);
  return round_up((size_t)N * (size_t)K * 4, 256);
}

// Backward workspace: [ones K | column-sum partials | s_w-scaled W^T [K, N] | dy^T | s_x-scaled xq^T | dw partials].
// The weight gradient is an [N, K] output with a contraction of M: few, very deep tiles.  Its
// contraction is therefore cut into `batches` chunks of `chunk` rows (a multiple of 32), each
// batch a matmul of its own in the same launch (GemmParams::batch_tiles_m), and the batches'
// outputs are added in order.  The split is chosen for the 148 SMs of the one device this library
// is built for, so that the layout (and aqt_workspace_bytes) needs no CUDA call.
struct BwdLayout {
  size_t ones, partial, wt, dyt, xt, dwp, total;
  int64_t batches, chunk, n_pad;  // batches == 1: chunk is the padded pitch of the transposed operands
};
BwdLayout bwd_layout(int64_t M, int64_t N, int64_t K) {
  BwdLayout L;
  L.n_pad = round_up((size_t)N, 128);
  const int64_t tiles = (L.n_pad / 128) * ceil_div(K, 256);
  int64_t batches = 148 / (tiles > 0 ? tiles : 1);
  if (batches > M / 512) batches = M / 512;  // a batch should still be some k-blocks deep
  if (batches < 2) {
    L.batches = 1;
    L.chunk = (M + 3) / 4 * 4;
    L.n_pad = N;
  } else {
    L.chunk = round_up((size_t)ceil_div(M, batches), kTrRows);
    L.batches = ceil_div(M, L.chunk);
  }
  L.ones = 0;
  L.partial = L.ones + round_up((size_t)K * 4, 256);
  // column-sum partials: one row of N per 128-row block of the transpose (or per 2048-row chunk of the stand-alone sum)
  L.wt = L.partial + round_up((size_t)(transpose_row_blocks(L.batches * L.chunk) + colsum_chunks(M)) * (size_t)N * 4, 256);
  L.dyt = L.wt + round_up((size_t)K * (size_t)N * 4, 256);
  L.xt = L.dyt + round_up((size_t)L.batches * L.n_pad * L.chunk * 4, 256);
  L.dwp = L.xt + round_up((size_t)L.batches * K * L.chunk * 4, 256);
  L.total = L.dwp + (L.batches > 1 ? round_up((size_t)L.batches * L.n_pad * K * 4, 256) : 0);
  return L;
}

// y[r][c] = sum_j a[r][j] * b[c][j] on the float kind of the GEMM (no scale, bias or activation).
// batches > 1: a holds `batches` stacked [rows / batches, depth] blocks, b as many stacked [cols, depth] blocks,
// and y receives the stacked [rows / batches, cols] products.
int float_gemm_nt(const float* a, int64_t lda, const float* b, int64_t rows, int64_t cols, int64_t depth, const float* ones, float* y,
                  int64_t ldy, cudaStream_t st, int64_t batches = 1) {
  GemmParams p;
  if (batches > 1) {
    p.batch_tiles_m = (int)(rows / batches / kBM);  // rows per batch are a multiple of the tile height
    p.batch_b_rows = (int)cols;
    p.b_rows = batches * cols;
  }
  p.s_x = nullptr;
  p.s_w = ones;
  p.bias = nullptr;
  p.residual = nullptr;
  p.acc_debug = nullptr;
  p.ldr = 0;
  p.residual_scale = 0.0f;
  p.s_x_kind = AQT_SCALE_TENSOR;
  p.act = AQT_ACT_NONE;
  p.M = (int)rows;
  p.N = (int)cols;
  p.K = (int)(4 * depth);
  p.kind = 1;
  p.a_pitch = 4 * lda;
  p.n_out = (int)cols;
  p.tiles_m = p.tiles_n = p.k_blocks = 0;
  p.small_acc = 0;
  return launch_qgemm(reinterpret_cast<const int8_t*>(a), b, false, y, ldy, p, st);
}

// True if the CTA-pair kernel with the row-quantizing epilogue takes the call: deep K, no GLU, int8
// codes out (4-bit codes stay in their containers), at most 16 column parts per row.
bool rowquant_pair_applies(int64_t M, int64_t N, int64_t K, int act, bool pack_out) {
  // (from K = 2048: at K = 1024 a tile's MMAs are shorter than its two epilogue passes, and the
  // two kernels are faster: 162 vs 209 us at 65 536 x 1024 -> 1024 with the fp32 output)
  if (pack_out || M <= kBM || K < 2048) return false;
  if (act != AQT_ACT_NONE && act != AQT_ACT_SWISH) return false;
  const int sms = sm_count() > 0 ? sm_count() : kDefaultSms;
  const int plan = rowquant_plan(M, N, K, sms);
  const int parts = rowquant_parts(plan, N);
  return parts % 2 == 0 && parts <= 16 && ceil_div(N, kGemmPlanBn[plan]) <= sms / 2;
}

int validate_matmul_shape(int64_t M, int64_t N, int64_t K, int bits_a, int bits_w, int act, int s_x_kind) {
  if (M < 0 || N < 0 || K <= 0) return AQT_ERR_BADARG;
  if (!bits_ok(bits_a) || !bits_ok(bits_w) || !act_ok(act)) return AQT_ERR_BADARG;
  if (s_x_kind != AQT_SCALE_ROW && s_x_kind != AQT_SCALE_TENSOR) return AQT_ERR_BADARG;
  if (K % 16 != 0 || N % 4 != 0 || (is_glu(act) && N % 8 != 0)) return AQT_ERR_BADARG;
  if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31) || M * N >= (1ll << 40)) return AQT_ERR_UNSUPPORTED;
  return AQT_OK;
}

int run_small_m(const void* xq, bool a_packed, const float* s_x, int s_x_kind, const void* wq, bool w_packed, const float* s_w,
                const float* bias, const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K, int act,
                float* y, int64_t ldy, int32_t* acc_debug, cudaStream_t st) {
  SmallParams sp;
  sp.xq = xq;
  sp.wq = wq;
  sp.s_x = s_x;
  sp.s_w = s_w;
  sp.bias = bias;
  sp.residual = residual;
  sp.y = y;
  sp.acc_debug = acc_debug;
  sp.ldr = ldr;
  sp.ldy = ldy;
  sp.residual_scale = residual_scale;
  sp.s_x_kind = s_x_kind;
  sp.act = act;
  sp.M = (int)M;
  sp.N = (int)N;
  sp.K = (int)K;
  sp.a_packed = a_packed ? 1 : 0;
  sp.w_packed = w_packed ? 1 : 0;
  return launch_small_m(sp, st);
}

// Codes already in int8 containers for A; B possibly packed.  ws holds B's unpacked copy.
int qmatmul_i8a(const int8_t* a_codes, const float* s_x, int s_x_kind, const void* wq, const float* s_w, const float* bias,
                const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K, int bits_a, int bits_w,
                int act, float* y, int64_t ldy, int32_t* acc_debug, uint8_t* ws, cudaStream_t st, int forced_plan = kPlanNone) {
  if (forced_plan == kPlanNone && small_m_applies(M, K)) {
    // a few rows: weight-bandwidth-bound kernel, packed weights read as they are
    return run_small_m(a_codes, false, s_x, s_x_kind, wq, is_packed(bits_w), s_w, bias, residual, ldr, residual_scale, M, N, K, act, y, ldy,
                       acc_debug, st);
  }
  // 4-bit weights: the weight-stationary kernel (K <= 512) sign-extends them itself in shared
  // memory after TMA staging; deeper K takes a one-off sign-extended copy in the workspace.
  const void* b_codes = wq;
  bool b_packed = false;
  if (is_packed(bits_w)) {
    const int sms = sm_count();
    if (sms <= 0) return AQT_ERR_CUDA;
    const int plan = forced_plan != kPlanNone ? forced_plan : plan_qgemm(GemmShape{M, N, K, act, 0, false}, sms);
    const bool ws_plan = plan == kPlanWs128E16 || plan == kPlanWs128E8;
    if (ws_plan && K % 32 == 0) {  // the packed rows must keep the 16-byte pitch bulk copies need
      b_packed = true;
    } else {
      int rc = launch_unpack_int4(reinterpret_cast<const uint8_t*>(wq), N * K / 2, reinterpret_cast<int8_t*>(ws), st);
      if (rc != AQT_OK) return rc;
      b_codes = ws;
    }
  }
  GemmParams p;
  p.s_x = s_x;
  p.s_w = s_w;
  p.bias = bias;
  p.residual = residual;
  p.acc_debug = acc_debug;
  p.ldr = ldr;
  p.residual_scale = residual_scale;
  p.s_x_kind = s_x_kind;
  p.act = act;
  p.M = (int)M;
  p.N = (int)N;
  p.K = (int)K;
  p.n_out = is_glu(act) ? (int)(N / 2) : (int)N;
  p.tiles_m = p.tiles_n = p.k_blocks = 0;
  // |acc| <= K * 2^(bits_a - 1) * 2^(bits_w - 1) for any codes the containers can hold
  p.small_acc = (K * (int64_t)(qmax_of(code_bits(bits_a)) + 1) * (qmax_of(code_bits(bits_w)) + 1) <= (1ll << 22)) ? 1 : 0;
  return launch_qgemm(a_codes, b_codes, b_packed, y, ldy, p, st, forced_plan);
}

// Workspace of aqt_ffn_fwd: [x on the device | y on the device | codes of x | scales | codes of u | scales | matmul scratch].
struct FfnLayout {
  size_t x, y, q1, s1, q2, s2, mm, total;
};
FfnLayout ffn_layout(int64_t M, int64_t d, int64_t ff, int bits_w1, int bits_w2) {
  FfnLayout L;
  L.x = 0;
  L.y = L.x + round_up((size_t)M * d * 4, 256);
  L.q1 = L.y + round_up((size_t)M * d * 4, 256);
  L.s1 = L.q1 + round_up((size_t)M * d, 256);
  L.q2 = L.s1 + round_up((size_t)M * 4, 256);
  L.s2 = L.q2 + round_up((size_t)M * ff, 256);
  L.mm = L.s2 + round_up((size_t)M * 4, 256);
  const size_t mm1 = round_up(ws_qmatmul(M, ff, d, 8, bits_w1), 256) + requant_exchange_bytes(M, ff);
  const size_t mm2 = ws_qmatmul(M, d, ff, 8, bits_w2);
  L.total = L.mm + round_up(mm1 > mm2 ? mm1 : mm2, 256);
  return L;
}

}  // namespace

extern "C" {

int aqt_version(void) { return AQT_VERSION; }

const char* aqt_status_string(int status) {
  switch (status) {
    case AQT_OK: return "ok";
    case AQT_ERR_BADARG: return "bad argument";
    case AQT_ERR_ALIGN: return "misaligned pointer or pitch";
    case AQT_ERR_UNSUPPORTED: return "unsupported device or size";
    case AQT_ERR_WORKSPACE: return "workspace missing or too small";
    case AQT_ERR_CUDA: return "CUDA call failed";
    case AQT_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

size_t aqt_workspace_bytes(int op, int64_t M, int64_t N, int64_t K, int bits_a, int bits_w) {
  if (M < 0 || N < 0 || K < 0) return 0;
  if (op == AQT_OP_QMATMUL) return ws_qmatmul(M, N, K, bits_a, bits_w);
  if (op == AQT_OP_LINEAR_FWD) return ws_linear(M, N, K, bits_w);
  if (op == AQT_OP_LINEAR_WEIGHT_ONLY) return ws_weight_only(0, N, K, AQT_FLOAT_TF32);
  if (op == AQT_OP_LINEAR_WEIGHT_ONLY_X2) return ws_weight_only(M, N, K, AQT_FLOAT_TF32X2);
  if (op == AQT_OP_LINEAR_BWD) return bwd_layout(M, N, K).total;
  if (op == AQT_OP_FFN_FWD) return ffn_layout(M, K, N, bits_w, bits_w).total;
  if (op == AQT_OP_QMATMUL_REQUANT) return round_up(ws_qmatmul(M, N, K, bits_a, bits_w), 256) + requant_exchange_bytes(M, N);
  return 0;
}

int aqt_quantize(const float* x, int64_t rows, int64_t cols, int64_t ld, int bits, int axis, int rounding, int pack,
                 void* q_out, float* scale_out, void* stream) {
  if (rows < 0 || cols < 0 || ld < cols || !quant_bits_ok(bits)) return AQT_ERR_BADARG;
  if (axis != AQT_AXIS_ROW && axis != AQT_AXIS_COL && axis != AQT_AXIS_TENSOR) return AQT_ERR_BADARG;
  if (rounding != AQT_ROUND_HALF_UP_FLOOR && rounding != AQT_ROUND_NEAREST_EVEN) return AQT_ERR_BADARG;
  if (pack != 0 && pack != 1) return AQT_ERR_BADARG;
  if (pack == 1 && (bits != 4 || cols % 2 != 0)) return AQT_ERR_BADARG;
  if (rows == 0 || cols == 0) return AQT_OK;
  if (x == nullptr || q_out == nullptr || scale_out == nullptr) return AQT_ERR_BADARG;
  if (!is_aligned(x, 4) || !is_aligned(scale_out, 4)) return AQT_ERR_ALIGN;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int qmax = qmax_of(bits);
  if (rounding == AQT_ROUND_HALF_UP_FLOOR) {
    return pack ? launch_quantize_axis<AQT_ROUND_HALF_UP_FLOOR, true>(x, rows, cols, ld, qmax, axis, q_out, scale_out, st)
                : launch_quantize_axis<AQT_ROUND_HALF_UP_FLOOR, false>(x, rows, cols, ld, qmax, axis, q_out, scale_out, st);
  }
  return pack ? launch_quantize_axis<AQT_ROUND_NEAREST_EVEN, true>(x, rows, cols, ld, qmax, axis, q_out, scale_out, st)
              : launch_quantize_axis<AQT_ROUND_NEAREST_EVEN, false>(x, rows, cols, ld, qmax, axis, q_out, scale_out, st);
}

int aqt_pack_int4(const int8_t* q, int64_t rows, int64_t cols, uint8_t* packed, void* stream) {
  if (rows < 0 || cols < 0 || cols % 2 != 0) return AQT_ERR_BADARG;
  if (rows == 0 || cols == 0) return AQT_OK;
  if (q == nullptr || packed == nullptr) return AQT_ERR_BADARG;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  return launch_pack_int4(q, rows * cols / 2, packed, reinterpret_cast<cudaStream_t>(stream));
}

int aqt_unpack_int4(const uint8_t* packed, int64_t rows, int64_t cols, int8_t* q, void* stream) {
  if (rows < 0 || cols < 0 || cols % 2 != 0) return AQT_ERR_BADARG;
  if (rows == 0 || cols == 0) return AQT_OK;
  if (q == nullptr || packed == nullptr) return AQT_ERR_BADARG;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  return launch_unpack_int4(packed, rows * cols / 2, q, reinterpret_cast<cudaStream_t>(stream));
}

static int qmatmul_entry(const void* xq, const float* s_x, int s_x_kind, const void* wq, const float* s_w, const float* bias,
                         const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K, int bits_a,
                         int bits_w, int act, float* y, int64_t ldy, int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                         void* stream, int forced_plan) {
  bits_w &= ~AQT_STATIC_WEIGHTS;
  int rc = validate_matmul_shape(M, N, K, bits_a, bits_w, act, s_x_kind);
  if (rc != AQT_OK) return rc;
  if (M == 0 || N == 0) return AQT_OK;
  const int64_t n_out = is_glu(act) ? N / 2 : N;
  if (xq == nullptr || s_x == nullptr || wq == nullptr || s_w == nullptr || y == nullptr) return AQT_ERR_BADARG;
  if (ldy < n_out || (residual != nullptr && ldr < n_out)) return AQT_ERR_BADARG;
  if (!is_aligned(xq, 16) || !is_aligned(wq, 16) || !is_aligned(y, 16) || !is_aligned(s_w, 16) || !is_aligned(s_x, 4) ||
      (bias != nullptr && !is_aligned(bias, 16)) || (residual != nullptr && !is_aligned(residual, 16)) ||
      (acc_debug != nullptr && !is_aligned(acc_debug, 4)))
    return AQT_ERR_ALIGN;
  if (ldy % 4 != 0 || (residual != nullptr && ldr % 4 != 0)) return AQT_ERR_ALIGN;
  const size_t need = ws_qmatmul(M, N, K, bits_a, bits_w);
  if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return AQT_ERR_WORKSPACE;
  if (need > 0 && !is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  rc = check_device();
  if (rc != AQT_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  if (forced_plan == kPlanNone && small_m_applies(M, K)) {
    return run_small_m(xq, is_packed(bits_a), s_x, s_x_kind, wq, is_packed(bits_w), s_w, bias, residual, ldr, residual_scale, M, N, K, act, y, ldy,
                       acc_debug, st);
  }
  const int8_t* a_codes = reinterpret_cast<const int8_t*>(xq);
  if (is_packed(bits_a)) {
    rc = launch_unpack_int4(reinterpret_cast<const uint8_t*>(xq), M * K / 2, reinterpret_cast<int8_t*>(ws), st);
    if (rc != AQT_OK) return rc;
    a_codes = reinterpret_cast<const int8_t*>(ws);
    ws += round_up((size_t)M * (size_t)K, 256);
  }
  return qmatmul_i8a(a_codes, s_x, s_x_kind, wq, s_w, bias, residual, ldr, residual_scale, M, N, K, bits_a, bits_w, act, y,
                     ldy, acc_debug, ws, st, forced_plan);
}

int aqt_qmatmul(const void* xq, const float* s_x, int s_x_kind, const void* wq, const float* s_w, const float* bias,
                const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K, int bits_a,
                int bits_w, int act, float* y, int64_t ldy, int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                void* stream) {
  return qmatmul_entry(xq, s_x, s_x_kind, wq, s_w, bias, residual, ldr, residual_scale, M, N, K, bits_a, bits_w, act, y, ldy, acc_debug,
                       workspace, workspace_bytes, stream, kPlanNone);
}

int aqt_qmatmul_with_plan(const char* plan, const void* xq, const float* s_x, int s_x_kind, const void* wq, const float* s_w,
                          const float* bias, const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N,
                          int64_t K, int bits_a, int bits_w, int act, float* y, int64_t ldy, int32_t* acc_debug, void* workspace,
                          size_t workspace_bytes, void* stream) {
  const int id = gemm_plan_by_name(plan);
  if (id == kPlanNone) return AQT_ERR_BADARG;
  return qmatmul_entry(xq, s_x, s_x_kind, wq, s_w, bias, residual, ldr, residual_scale, M, N, K, bits_a, bits_w, act, y, ldy, acc_debug,
                       workspace, workspace_bytes, stream, id);
}

int aqt_plan_qmatmul(int64_t M, int64_t N, int64_t K, int bits_a, int bits_w, int act, int float_kind, int sm_count_or_0,
                     char* name_out, size_t name_bytes) {
  if (name_out == nullptr || name_bytes == 0 || M <= 0 || N <= 0 || K <= 0 || !act_ok(act)) return AQT_ERR_BADARG;
  if (!float_kind && (!bits_ok(bits_a) || !bits_ok(bits_w))) return AQT_ERR_BADARG;
  int sms = sm_count_or_0;
  if (sms <= 0) sms = sm_count();
  if (sms <= 0) sms = kDefaultSms;
  const char* name;
  if (!float_kind && small_m_applies(M, K)) {
    name = "small_m";
  } else {
    name = gemm_plan_name(plan_qgemm(GemmShape{M, N, float_kind ? 4 * K : K, act, float_kind ? 1 : 0, false}, sms));
  }
  if (strlen(name) + 1 > name_bytes) return AQT_ERR_BADARG;
  memcpy(name_out, name, strlen(name) + 1);
  return AQT_OK;
}

int aqt_qmatmul_requant(const void* xq, const float* s_x, int s_x_kind, const void* wq, const float* s_w, const float* bias,
                        const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K, int bits_a,
                        int bits_w, int act, int bits_out, int rounding, int pack_out, void* q_out, float* s_out, float* y,
                        int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
  const int static_w = (bits_w & AQT_STATIC_WEIGHTS) ? 1 : 0;
  bits_w &= ~AQT_STATIC_WEIGHTS;
  int rc = validate_matmul_shape(M, N, K, bits_a, bits_w, act, s_x_kind);
  if (rc != AQT_OK) return rc;
  if (!quant_bits_ok(bits_out) || (pack_out != 0 && pack_out != 1) || (pack_out == 1 && bits_out != 4)) return AQT_ERR_BADARG;
  if (rounding != AQT_ROUND_HALF_UP_FLOOR && rounding != AQT_ROUND_NEAREST_EVEN) return AQT_ERR_BADARG;
  const int64_t n_out = is_glu(act) ? N / 2 : N;
  if (n_out % (pack_out ? 32 : 16) != 0) return AQT_ERR_BADARG;  // rows of codes keep a 16-byte pitch
  if (residual != nullptr && y == nullptr) return AQT_ERR_BADARG;
  if (M == 0 || N == 0) return AQT_OK;
  if (xq == nullptr || s_x == nullptr || wq == nullptr || s_w == nullptr || q_out == nullptr || s_out == nullptr) return AQT_ERR_BADARG;
  if (y != nullptr && (ldy < n_out || ldy % 4 != 0)) return AQT_ERR_BADARG;
  if (residual != nullptr && (ldr < n_out || ldr % 4 != 0)) return AQT_ERR_BADARG;
  if (!is_aligned(xq, 16) || !is_aligned(wq, 16) || !is_aligned(q_out, 16) || !is_aligned(s_w, 16) || !is_aligned(s_x, 4) ||
      !is_aligned(s_out, 4) || (y != nullptr && !is_aligned(y, 16)) || (bias != nullptr && !is_aligned(bias, 16)) ||
      (residual != nullptr && !is_aligned(residual, 16)))
    return AQT_ERR_ALIGN;
  const size_t mm_bytes = round_up(ws_qmatmul(M, N, K, bits_a, bits_w), 256);
  const size_t need = mm_bytes + requant_exchange_bytes(M, N);
  if (workspace == nullptr || workspace_bytes < need) return AQT_ERR_WORKSPACE;
  if (!is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  rc = check_device();
  if (rc != AQT_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);

  if (!requant_applies(M, N, K, act, y != nullptr, pack_out != 0) && rowquant_pair_applies(M, N, K, act, pack_out != 0)) {
    // Deep K (the second feed-forward layers): the CTA-pair kernel with the row-quantizing epilogue
    const int8_t* a_codes = reinterpret_cast<const int8_t*>(xq);
    if (is_packed(bits_a)) {
      rc = launch_unpack_int4(reinterpret_cast<const uint8_t*>(xq), M * K / 2, reinterpret_cast<int8_t*>(ws), st);
      if (rc != AQT_OK) return rc;
      a_codes = reinterpret_cast<const int8_t*>(ws);
      ws += round_up((size_t)M * (size_t)K, 256);
    }
    const void* b_codes = wq;
    if (is_packed(bits_w)) {
      rc = launch_unpack_int4(reinterpret_cast<const uint8_t*>(wq), N * K / 2, reinterpret_cast<int8_t*>(ws), st);
      if (rc != AQT_OK) return rc;
      b_codes = ws;
    }
    GemmParams p;
    p.s_x = s_x;
    p.s_w = s_w;
    p.bias = bias;
    p.residual = residual;
    p.acc_debug = nullptr;
    p.ldr = ldr;
    p.residual_scale = residual_scale;
    p.s_x_kind = s_x_kind;
    p.act = act;
    p.M = (int)M;
    p.N = (int)N;
    p.K = (int)K;
    p.n_out = (int)N;
    p.tiles_m = p.tiles_n = p.k_blocks = 0;
    p.small_acc = (K * (int64_t)(qmax_of(code_bits(bits_a)) + 1) * (qmax_of(code_bits(bits_w)) + 1) <= (1ll << 22)) ? 1 : 0;
    p.q_out = reinterpret_cast<uint8_t*>(q_out);
    p.s_out = s_out;
    p.exchange = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(workspace) + mm_bytes);
    p.generation = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(workspace) + mm_bytes + requant_exchange_bytes(M, N) - (size_t)kMaxGroups * 4);
    p.tag = next_launch_tag();
    p.qmax_out = qmax_of(bits_out);
    p.rounding = rounding;
    p.has_y = y != nullptr ? 1 : 0;
    const int sms = sm_count();
    if (sms <= 0) return AQT_ERR_CUDA;
    return launch_qgemm_rowquant(rowquant_plan(M, N, K, sms), a_codes, b_codes, y, ldy, p, st);
  }
  if (!requant_applies(M, N, K, act, y != nullptr, pack_out != 0)) {
    // Shapes the fused kernels do not take: the two steps one after the other, through y.
    if (y == nullptr) return AQT_ERR_UNSUPPORTED;
    rc = aqt_qmatmul(xq, s_x, s_x_kind, wq, s_w, bias, residual, ldr, residual_scale, M, N, K, bits_a, bits_w, act, y, ldy, nullptr,
                     workspace, mm_bytes, stream);
    if (rc != AQT_OK) return rc;
    return aqt_quantize(y, M, n_out, ldy, bits_out, AQT_AXIS_ROW, rounding, pack_out, q_out, s_out, stream);
  }

  const int8_t* a_codes = reinterpret_cast<const int8_t*>(xq);
  if (is_packed(bits_a)) {
    rc = launch_unpack_int4(reinterpret_cast<const uint8_t*>(xq), M * K / 2, reinterpret_cast<int8_t*>(ws), st);
    if (rc != AQT_OK) return rc;
    a_codes = reinterpret_cast<const int8_t*>(ws);
    ws += round_up((size_t)M * (size_t)K, 256);
  }
  const void* b_codes = wq;
  bool b_packed = false;
  if (is_packed(bits_w)) {
    if (K % 32 == 0 && K <= 512) {  // the deep-K form (512 < K <= 1024) has no room to unpack in shared memory
      b_packed = true;
    } else {
      rc = launch_unpack_int4(reinterpret_cast<const uint8_t*>(wq), N * K / 2, reinterpret_cast<int8_t*>(ws), st);
      if (rc != AQT_OK) return rc;
      b_codes = ws;
    }
  }
  RequantParams rp;
  GemmParams& p = rp.g;
  p.s_x = s_x;
  p.s_w = s_w;
  p.bias = bias;
  p.residual = residual;
  p.acc_debug = nullptr;
  p.ldr = ldr;
  p.residual_scale = residual_scale;
  p.s_x_kind = s_x_kind;
  p.act = act;
  p.M = (int)M;
  p.N = (int)N;
  p.K = (int)K;
  p.n_out = (int)n_out;
  p.tiles_m = p.tiles_n = p.k_blocks = 0;
  p.small_acc = (K * (int64_t)(qmax_of(code_bits(bits_a)) + 1) * (qmax_of(code_bits(bits_w)) + 1) <= (1ll << 22)) ? 1 : 0;
  p.static_w = (static_w && (!is_packed(bits_w) || b_packed)) ? 1 : 0;  // not for weights unpacked into the workspace just now
  rp.q_out = nullptr;
  rp.s_out = s_out;
  rp.exchange = nullptr;
  rp.qmax_out = qmax_of(bits_out);
  rp.rounding = rounding;
  rp.pack_out = pack_out;
  return launch_requant(a_codes, b_codes, b_packed, q_out, y, ldy, rp, reinterpret_cast<uint8_t*>(workspace) + mm_bytes, st);
}

int aqt_linear_fwd(const float* x, int64_t ldx, const void* wq, const float* s_w, const float* bias, const float* residual,
                   int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K, int bits_a, int bits_w,
                   int a_scale_kind, int rounding, int act, float* y, int64_t ldy, void* workspace, size_t workspace_bytes,
                   void* stream) {
  bits_w &= ~AQT_STATIC_WEIGHTS;
  int rc = validate_matmul_shape(M, N, K, bits_a, bits_w, act, a_scale_kind);
  if (rc != AQT_OK) return rc;
  if (rounding != AQT_ROUND_HALF_UP_FLOOR && rounding != AQT_ROUND_NEAREST_EVEN) return AQT_ERR_BADARG;
  if (!quant_bits_ok(bits_a)) return AQT_ERR_BADARG;  // the width the activations are quantized to
  if (M == 0 || N == 0) return AQT_OK;
  const int64_t n_out = is_glu(act) ? N / 2 : N;
  if (x == nullptr || wq == nullptr || s_w == nullptr || y == nullptr) return AQT_ERR_BADARG;
  if (ldx < K || ldy < n_out || (residual != nullptr && ldr < n_out)) return AQT_ERR_BADARG;
  if (!is_aligned(x, 4) || !is_aligned(wq, 16) || !is_aligned(y, 16) || !is_aligned(s_w, 16) ||
      (bias != nullptr && !is_aligned(bias, 16)) || (residual != nullptr && !is_aligned(residual, 16)))
    return AQT_ERR_ALIGN;
  if (ldy % 4 != 0 || (residual != nullptr && ldr % 4 != 0)) return AQT_ERR_ALIGN;
  const size_t need = ws_linear(M, N, K, bits_w);
  if (workspace == nullptr || workspace_bytes < need) return AQT_ERR_WORKSPACE;
  if (!is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  rc = check_device();
  if (rc != AQT_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  int8_t* codes = reinterpret_cast<int8_t*>(ws);
  float* s_x = reinterpret_cast<float*>(ws + round_up((size_t)M * (size_t)K, 256));
  uint8_t* ws_mm = ws + round_up((size_t)M * (size_t)K, 256) + round_up((size_t)M * 4, 256);
  // Step 1 (Fig. 2): dynamic quantization of the activations over K; 4-bit codes stay in int8
  // containers between the two kernels, which is what the figure's cast produces.
  const int axis = a_scale_kind == AQT_SCALE_ROW ? AQT_AXIS_ROW : AQT_AXIS_TENSOR;
  rc = aqt_quantize(x, M, K, ldx, bits_a, axis, rounding, 0, codes, s_x, stream);
  if (rc != AQT_OK) return rc;
  // Step 2: integer matmul + de-quantizing epilogue.
  return qmatmul_i8a(codes, s_x, a_scale_kind, wq, s_w, bias, residual, ldr, residual_scale, M, N, K, bits_a, bits_w, act, y,
                     ldy, nullptr, ws_mm, st);
}

int aqt_linear_fwd_host(const float* x, int x_on_host, const void* wq, const float* s_w, const float* bias, int64_t M,
                        int64_t N, int64_t K, int bits_a, int bits_w, int a_scale_kind, int rounding, int act, float* y,
                        int y_on_host, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = validate_matmul_shape(M, N, K, bits_a, bits_w, act, a_scale_kind);
  if (rc != AQT_OK) return rc;
  if (M == 0 || N == 0) return AQT_OK;
  if (x == nullptr || y == nullptr) return AQT_ERR_BADARG;
  const int64_t n_out = is_glu(act) ? N / 2 : N;
  const size_t layer = round_up(ws_linear(M, N, K, bits_w), 256);
  const size_t xb = x_on_host ? round_up((size_t)M * K * 4, 256) : 0;
  const size_t yb = y_on_host ? round_up((size_t)M * n_out * 4, 256) : 0;
  if (workspace == nullptr || workspace_bytes < layer + xb + yb) return AQT_ERR_WORKSPACE;
  if (!is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const float* x_dev = x;
  float* y_dev = y;
  if (x_on_host) {
    float* xd = reinterpret_cast<float*>(ws + layer);
    AQT_RETURN_IF_CUDA(cudaMemcpyAsync(xd, x, (size_t)M * K * 4, cudaMemcpyHostToDevice, st));
    x_dev = xd;
  }
  if (y_on_host) y_dev = reinterpret_cast<float*>(ws + layer + xb);
  rc = aqt_linear_fwd(x_dev, K, wq, s_w, bias, nullptr, 0, 0.0f, M, N, K, bits_a, bits_w, a_scale_kind, rounding, act, y_dev,
                      n_out, ws, layer, stream);
  if (rc != AQT_OK) return rc;
  if (y_on_host) AQT_RETURN_IF_CUDA(cudaMemcpyAsync(y, y_dev, (size_t)M * n_out * 4, cudaMemcpyDeviceToHost, st));
  return AQT_OK;
}

int aqt_ffn_fwd(const float* x, int x_on_host, const void* w1q, const float* s_w1, const float* bias1, int bits_w1,
                const void* w2q, const float* s_w2, const float* bias2, int bits_w2, int64_t M, int64_t d, int64_t ff,
                int bits_a, int rounding, int act, float* y, int y_on_host, void* workspace, size_t workspace_bytes,
                void* stream) {
  const int static_flag = (bits_w1 | bits_w2) & AQT_STATIC_WEIGHTS;
  bits_w1 &= ~AQT_STATIC_WEIGHTS;
  bits_w2 &= ~AQT_STATIC_WEIGHTS;
  if (M < 0 || d <= 0 || ff <= 0 || !quant_bits_ok(bits_a) || !bits_ok(bits_w1) || !bits_ok(bits_w2)) return AQT_ERR_BADARG;
  if (act != AQT_ACT_NONE && act != AQT_ACT_SWISH) return AQT_ERR_BADARG;
  if (rounding != AQT_ROUND_HALF_UP_FLOOR && rounding != AQT_ROUND_NEAREST_EVEN) return AQT_ERR_BADARG;
  if (M == 0) return AQT_OK;
  if (x == nullptr || y == nullptr || w1q == nullptr || w2q == nullptr || s_w1 == nullptr || s_w2 == nullptr) return AQT_ERR_BADARG;
  const FfnLayout L = ffn_layout(M, d, ff, bits_w1, bits_w2);
  if (workspace == nullptr || workspace_bytes < L.total) return AQT_ERR_WORKSPACE;
  if (!is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  if (!requant_applies(M, ff, d, act, false, false)) return AQT_ERR_UNSUPPORTED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const float* x_dev = x;
  float* y_dev = y;
  if (x_on_host) {
    AQT_RETURN_IF_CUDA(cudaMemcpyAsync(ws + L.x, x, (size_t)M * d * 4, cudaMemcpyHostToDevice, st));
    x_dev = reinterpret_cast<const float*>(ws + L.x);
  }
  if (y_on_host) y_dev = reinterpret_cast<float*>(ws + L.y);
  int8_t* q1 = reinterpret_cast<int8_t*>(ws + L.q1);
  float* s1 = reinterpret_cast<float*>(ws + L.s1);
  int8_t* q2 = reinterpret_cast<int8_t*>(ws + L.q2);
  float* s2 = reinterpret_cast<float*>(ws + L.s2);
  const size_t mm_bytes = L.total - L.mm;
  // Fig. 2 on the input rows; first matmul with the rows of u = act(W1 x) quantized in its epilogue
  // (4-bit codes stay in int8 containers between the kernels); second matmul.
  rc = aqt_quantize(x_dev, M, d, d, bits_a, AQT_AXIS_ROW, rounding, 0, q1, s1, stream);
  if (rc != AQT_OK) return rc;
  const int bits_mm = bits_a == 8 ? 8 : AQT_BITS_4_UNPACKED;
  rc = aqt_qmatmul_requant(q1, s1, AQT_SCALE_ROW, w1q, s_w1, bias1, nullptr, 0, 0.0f, M, ff, d, bits_mm, bits_w1 | static_flag, act, bits_a, rounding, 0,
                           q2, s2, nullptr, 0, ws + L.mm, mm_bytes, stream);
  if (rc != AQT_OK) return rc;
  rc = aqt_qmatmul(q2, s2, AQT_SCALE_ROW, w2q, s_w2, bias2, nullptr, 0, 0.0f, M, d, ff, bits_mm, bits_w2, AQT_ACT_NONE, y_dev, d, nullptr,
                   ws + L.mm, mm_bytes, stream);
  if (rc != AQT_OK) return rc;
  if (y_on_host) AQT_RETURN_IF_CUDA(cudaMemcpyAsync(y, y_dev, (size_t)M * d * 4, cudaMemcpyDeviceToHost, st));
  return AQT_OK;
}

int aqt_linear_fwd_weight_only(const float* x, int64_t ldx, const void* wq, const float* s_w, const float* bias,
                               const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N, int64_t K,
                               int bits_w, int precision, int act, float* y, int64_t ldy, void* workspace,
                               size_t workspace_bytes, void* stream) {
  if (M < 0 || N < 0 || K <= 0 || !bits_ok(bits_w) || !act_ok(act)) return AQT_ERR_BADARG;
  if (precision != AQT_FLOAT_TF32 && precision != AQT_FLOAT_TF32X2) return AQT_ERR_BADARG;
  if (K % 4 != 0 || N % 4 != 0 || (is_glu(act) && N % 8 != 0)) return AQT_ERR_BADARG;
  if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 28) || M * N >= (1ll << 40)) return AQT_ERR_UNSUPPORTED;
  if (M == 0 || N == 0) return AQT_OK;
  const int64_t n_out = is_glu(act) ? N / 2 : N;
  if (x == nullptr || wq == nullptr || s_w == nullptr || y == nullptr) return AQT_ERR_BADARG;
  if (ldx < K || ldy < n_out || (residual != nullptr && ldr < n_out)) return AQT_ERR_BADARG;
  if (!is_aligned(x, 16) || !is_aligned(wq, 16) || !is_aligned(y, 16) || !is_aligned(s_w, 16) ||
      (bias != nullptr && !is_aligned(bias, 16)) || (residual != nullptr && !is_aligned(residual, 16)))
    return AQT_ERR_ALIGN;
  if (ldx % 4 != 0 || ldy % 4 != 0 || (residual != nullptr && ldr % 4 != 0)) return AQT_ERR_ALIGN;
  const size_t need = ws_weight_only(M, N, K, precision);
  if (workspace == nullptr || workspace_bytes < need) return AQT_ERR_WORKSPACE;
  if (!is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // the weights converted to float (Section 4.1): the codes as binary32 integers, once per call;
  // the channel scales stay outside the sum and are applied to the accumulators.
  float* w_f = reinterpret_cast<float*>(workspace);
  const float* a_f = x;
  int64_t k_mm = K, a_pitch = 4 * ldx;
  if (precision == AQT_FLOAT_TF32X2) {
    // x = hi + lo with hi a tf32 value: one matmul over [hi | lo] against [w | w]
    float* x2 = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace) + round_up((size_t)N * (size_t)K * 8, 256));
    rc = launch_codes_to_float_twice(wq, is_packed(bits_w), N, K, w_f, st);
    if (rc != AQT_OK) return rc;
    rc = launch_split_hi_lo(x, ldx, M, K, x2, st);
    if (rc != AQT_OK) return rc;
    a_f = x2;
    k_mm = 2 * K;
    a_pitch = 8 * K;
  } else {
    rc = launch_codes_to_float(wq, is_packed(bits_w), N * K, w_f, st);
    if (rc != AQT_OK) return rc;
  }
  GemmParams p;
  p.s_x = nullptr;
  p.s_w = s_w;
  p.bias = bias;
  p.residual = residual;
  p.acc_debug = nullptr;
  p.ldr = ldr;
  p.residual_scale = residual_scale;
  p.s_x_kind = AQT_SCALE_TENSOR;
  p.act = act;
  p.M = (int)M;
  p.N = (int)N;
  p.K = (int)(4 * k_mm);
  p.kind = 1;
  p.a_pitch = a_pitch;
  p.n_out = (int)n_out;
  p.tiles_m = p.tiles_n = p.k_blocks = 0;
  p.small_acc = 0;
  return launch_qgemm(reinterpret_cast<const int8_t*>(a_f), w_f, false, y, ldy, p, st);
}

int aqt_linear_bwd(const float* dy, int64_t lddy, const void* xq, const float* s_x, int s_x_kind, int bits_a, const void* wq,
                   const float* s_w, int bits_w, int64_t M, int64_t N, int64_t K, float* dx, int64_t lddx, float* dw, int64_t lddw,
                   float* dbias, void* workspace, size_t workspace_bytes, void* stream) {
  if (M < 0 || N < 0 || K <= 0 || !bits_ok(bits_a) || !bits_ok(bits_w)) return AQT_ERR_BADARG;
  if (s_x_kind != AQT_SCALE_ROW && s_x_kind != AQT_SCALE_TENSOR) return AQT_ERR_BADARG;
  if (K % 4 != 0 || N % 4 != 0) return AQT_ERR_BADARG;
  // M and N are row counts of the transposing prepasses, whose 128-row blocks are a grid's y extent (at most 65 535)
  if (M >= (1ll << 23) || N >= (1ll << 23) || K >= (1ll << 28) || M * N >= (1ll << 40)) return AQT_ERR_UNSUPPORTED;
  if (M == 0 || N == 0) return AQT_OK;
  if (dy == nullptr || lddy < N) return AQT_ERR_BADARG;
  if (dx != nullptr && (wq == nullptr || s_w == nullptr || lddx < K)) return AQT_ERR_BADARG;
  if (dw != nullptr && (xq == nullptr || s_x == nullptr || lddw < K)) return AQT_ERR_BADARG;
  if (!is_aligned(dy, 16) || lddy % 4 != 0) return AQT_ERR_ALIGN;
  if (dx != nullptr && (!is_aligned(dx, 16) || lddx % 4 != 0)) return AQT_ERR_ALIGN;
  if (dw != nullptr && (!is_aligned(dw, 16) || lddw % 4 != 0)) return AQT_ERR_ALIGN;
  if (dbias != nullptr && !is_aligned(dbias, 4)) return AQT_ERR_ALIGN;
  if ((dx != nullptr && !is_aligned(wq, 16)) || (dw != nullptr && !is_aligned(xq, 16))) return AQT_ERR_ALIGN;
  const BwdLayout L = bwd_layout(M, N, K);
  if (workspace == nullptr || workspace_bytes < L.total) return AQT_ERR_WORKSPACE;
  if (!is_aligned(workspace, 256)) return AQT_ERR_ALIGN;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  float* ones = reinterpret_cast<float*>(ws + L.ones);
  rc = launch_fill_f32(ones, K, 1.0f, st);
  if (rc != AQT_OK) return rc;
  if (dbias != nullptr && dw == nullptr) {  // with dw the column sums come out of the transpose of dy
    rc = launch_colsum(dy, lddy, M, N, reinterpret_cast<float*>(ws + L.partial), dbias, st);
    if (rc != AQT_OK) return rc;
  }
  if (dx != nullptr) {
    // dx = dy . (s_w wq): rows m, columns k, contraction n
    float* wt = reinterpret_cast<float*>(ws + L.wt);
    rc = launch_transpose_scale_codes(wq, is_packed(bits_w), s_w, true, N, K, wt, N, N, K, st);
    if (rc != AQT_OK) return rc;
    rc = float_gemm_nt(dy, lddy, wt, M, K, N, ones, dx, lddx, st);
    if (rc != AQT_OK) return rc;
  }
  if (dw != nullptr) {
    // dw = dy^T . (s_x xq): rows n, columns k, contraction m (padded with zeros), cut into L.batches chunks
    float* dyt = reinterpret_cast<float*>(ws + L.dyt);
    float* xt = reinterpret_cast<float*>(ws + L.xt);
    const int64_t m_pad = L.batches * L.chunk;
    rc = launch_transpose_f32(dy, lddy, M, N, dyt, m_pad, L.chunk, L.n_pad, dbias != nullptr ? reinterpret_cast<float*>(ws + L.partial) : nullptr,
                              dbias, st);
    if (rc != AQT_OK) return rc;
    rc = launch_transpose_scale_codes(xq, is_packed(bits_a), s_x, s_x_kind == AQT_SCALE_ROW, M, K, xt, m_pad, L.chunk, K, st);
    if (rc != AQT_OK) return rc;
    if (L.batches == 1) {
      rc = float_gemm_nt(dyt, L.chunk, xt, N, K, L.chunk, ones, dw, lddw, st);
      if (rc != AQT_OK) return rc;
    } else {
      float* dwp = reinterpret_cast<float*>(ws + L.dwp);
      rc = float_gemm_nt(dyt, L.chunk, xt, L.batches * L.n_pad, K, L.chunk, ones, dwp, K, st, L.batches);
      if (rc != AQT_OK) return rc;
      rc = launch_sum_batches(dwp, L.batches, L.n_pad, N, K, dw, lddw, st);
      if (rc != AQT_OK) return rc;
    }
  }
  return AQT_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant: the scratch lives in the library image.

// Sign-extended weight codes of the call in flight.  This name is only a host-side handle in
// host code; its device address comes from cudaGetSymbolAddress (noalloc_scratch_address).
static __device__ __align__(256) uint8_t g_noalloc_weight_scratch[AQT_NOALLOC_MAX_WEIGHT_BYTES];

// Device address of the scratch array on the current device, looked up once per device.
static int noalloc_scratch_address(uint8_t** out) {
  constexpr int kMaxDevices = 64;
  static uint8_t* cached[kMaxDevices] = {nullptr};
  int dev = 0;
  AQT_RETURN_IF_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return AQT_ERR_UNSUPPORTED;
  if (cached[dev] == nullptr) {
    void* ptr = nullptr;
    AQT_RETURN_IF_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_weight_scratch));
    if (ptr == nullptr) return AQT_ERR_CUDA;
    cached[dev] = reinterpret_cast<uint8_t*>(ptr);
  }
  *out = cached[dev];
  return AQT_OK;
}

int aqt_qmatmul_w4_noalloc(const int8_t* xq, const float* s_x, int s_x_kind, const uint8_t* wq_packed, const float* s_w,
                           const float* bias, const float* residual, int64_t ldr, float residual_scale, int64_t M, int64_t N,
                           int64_t K, int act, float* y, int64_t ldy, void* stream) {
  int rc = validate_matmul_shape(M, N, K, 8, 4, act, s_x_kind);
  if (rc != AQT_OK) return rc;
  if (M == 0 || N == 0) return AQT_OK;
  if ((uint64_t)N * (uint64_t)K > (uint64_t)AQT_NOALLOC_MAX_WEIGHT_BYTES) {
    if (debug_enabled())
      fprintf(stderr, "[aqt] aqt_qmatmul_w4_noalloc: N*K = %lld exceeds the built-in scratch of %u bytes\n", (long long)(N * K),
              AQT_NOALLOC_MAX_WEIGHT_BYTES);
    return AQT_ERR_UNSUPPORTED;
  }
  const int64_t n_out = is_glu(act) ? N / 2 : N;
  if (xq == nullptr || s_x == nullptr || wq_packed == nullptr || s_w == nullptr || y == nullptr) return AQT_ERR_BADARG;
  if (ldy < n_out || (residual != nullptr && ldr < n_out)) return AQT_ERR_BADARG;
  if (!is_aligned(xq, 16) || !is_aligned(wq_packed, 16) || !is_aligned(y, 16) || !is_aligned(s_w, 16) || !is_aligned(s_x, 4) ||
      (bias != nullptr && !is_aligned(bias, 16)) || (residual != nullptr && !is_aligned(residual, 16)))
    return AQT_ERR_ALIGN;
  if (ldy % 4 != 0 || (residual != nullptr && ldr % 4 != 0)) return AQT_ERR_ALIGN;
  rc = check_device();
  if (rc != AQT_OK) return rc;
  uint8_t* scratch = nullptr;
  rc = noalloc_scratch_address(&scratch);
  if (rc != AQT_OK) return rc;
  // qmatmul_i8a unpacks the weights into `scratch` (all N*K bytes it later reads) and runs the GEMM.
  return qmatmul_i8a(xq, s_x, s_x_kind, wq_packed, s_w, bias, residual, ldr, residual_scale, M, N, K, 8, 4, act, y, ldy, nullptr,
                     scratch, reinterpret_cast<cudaStream_t>(stream));
}

int aqt_selftest_bounded_wait(uint64_t limit_ns, int* gave_up_dev, void* stream) {
  if (gave_up_dev == nullptr || limit_ns == 0 || limit_ns > 1000000000ull) return AQT_ERR_BADARG;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  bounded_wait_selftest_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(limit_ns, gave_up_dev);
  return AQT_LAUNCH_STATUS();
}

// Nothing but special-function work: eight independent chains of 2^x and reciprocal per thread.
__global__ void __launch_bounds__(256) sfu_rate_kernel(int iterations, float* sink) {
  float v[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = 0.25f + 0.01f * (float)((threadIdx.x + j) & 15);
  for (int i = 0; i < iterations; ++i) {
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = rcp_approx(1.0f + ex2_approx(v[j]));
  }
  float acc = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) acc += v[j];
  if (acc == 12345.0f) *sink = acc;  // never true: keeps the chains alive
}

int aqt_selftest_sfu_rate(int iterations, float* sink_dev, int64_t* ops_out, void* stream) {
  if (iterations <= 0 || iterations > (1 << 20) || sink_dev == nullptr || ops_out == nullptr) return AQT_ERR_BADARG;
  int rc = check_device();
  if (rc != AQT_OK) return rc;
  const int sms = sm_count();
  if (sms <= 0) return AQT_ERR_CUDA;
  const int ctas = sms * 8;
  sfu_rate_kernel<<<ctas, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(iterations, sink_dev);
  *ops_out = (int64_t)ctas * 256 * iterations * 16;
  return AQT_LAUNCH_STATUS();
}

int aqt_device_status(void* stream, int* status_out) {
  if (status_out == nullptr) return AQT_ERR_BADARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  AQT_RETURN_IF_CUDA(cudaStreamSynchronize(st));
  int v = 0;
  AQT_RETURN_IF_CUDA(cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)));
  if (v != 0) {
    const int zero = 0;
    AQT_RETURN_IF_CUDA(cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)));
  }
  *status_out = v;
  return AQT_OK;
}

}  // extern "C"
