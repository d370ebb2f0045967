// Shared host/device helpers of the quantized-linear library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <atomic>

#include "../../include/aqt.h"

namespace aqt {

// Device status word: kernels record a bounded wait that ran out here; the host reads and
// clears it in aqt_device_status().  One word per loaded library image and device.
__device__ int g_device_status = 0;

// With AQT_DEBUG set in the environment, failing CUDA calls are described on stderr.
inline bool debug_enabled() {
  static int on = -1;
  if (on < 0) on = (getenv("AQT_DEBUG") != nullptr) ? 1 : 0;
  return on == 1;
}
inline int cuda_fail(cudaError_t e, const char* what, int line) {
  if (debug_enabled()) fprintf(stderr, "[aqt] %s (line %d): %s\n", what, line, cudaGetErrorString(e));
  return AQT_ERR_CUDA;
}

#define AQT_RETURN_IF_CUDA(expr)                                      \
  do {                                                                \
    cudaError_t _e = (expr);                                          \
    if (_e != cudaSuccess) return cuda_fail(_e, #expr, __LINE__);     \
  } while (0)

// Status of the launch just issued.
#define AQT_LAUNCH_STATUS() (aqt::launch_status(__LINE__))
inline int launch_status(int line) {
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? AQT_OK : cuda_fail(e, "kernel launch", line);
}

// Properties of the current device, looked up once per device ordinal.  Host threads may race on
// the first lookup; both then store the same values.
constexpr int kMaxDevices = 64;
struct DeviceInfo {
  int ordinal;
  int sms;       // multiprocessors
  int cc_major;  // compute capability, major
};
inline int current_device_info(DeviceInfo* out) {
  static std::atomic<int> sms[kMaxDevices];
  static std::atomic<int> cc[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return AQT_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return AQT_ERR_UNSUPPORTED;
  int n = sms[dev].load(std::memory_order_acquire);
  if (n == 0) {
    int major = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return AQT_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return AQT_ERR_CUDA;
    cc[dev].store(major, std::memory_order_relaxed);
    sms[dev].store(n, std::memory_order_release);
  }
  out->ordinal = dev;
  out->sms = n;
  out->cc_major = cc[dev].load(std::memory_order_relaxed);
  return AQT_OK;
}
// Multiprocessors of the current device; 0 if there is none (callers that only plan then assume
// the 148 of the one part this library is built for).
inline int sm_count() {
  DeviceInfo d;
  return current_device_info(&d) == AQT_OK ? d.sms : 0;
}
constexpr int kDefaultSms = 148;

// Opt a kernel into `bytes` of dynamic shared memory, once per device (the attribute belongs to
// the function as loaded on one device).  `done` is one mask per kernel instantiation.
template <class Kernel>
inline int ensure_dynamic_smem(Kernel kernel, int bytes, std::atomic<uint64_t>& done) {
  DeviceInfo d;
  int rc = current_device_info(&d);
  if (rc != AQT_OK) return rc;
  const uint64_t bit = 1ull << d.ordinal;
  if (done.load(std::memory_order_acquire) & bit) return AQT_OK;
  AQT_RETURN_IF_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  done.fetch_or(bit, std::memory_order_release);
  return AQT_OK;
}

// Launch with the programmatic-stream-serialization attribute (see grid_dependency_wait), optionally
// as thread-block clusters of `cluster` CTAs.
template <class... KArgs, class... Args>
inline int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, unsigned cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  AQT_RETURN_IF_CUDA(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
  return launch_status(__LINE__);
}

// Overrides of the kernel choice for tuning runs.  They exist only in builds made with
// -DAQT_TUNING; the shipped library never reads the environment to pick a kernel.
inline const char* tuning_env(const char* name) {
#ifdef AQT_TUNING
  return getenv(name);
#else
  (void)name;
  return nullptr;
#endif
}

inline bool is_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

__host__ __device__ inline int qmax_of(int bits) { return bits == 8 ? 127 : 7; }

// Per-scale constants of the quantizer of Fig. 2 for one reduced group (row, column or tensor).
// The figure divides every element by the scale in binary32.  The quotient x / s is formed here
// as the correctly rounded binary32 value by one multiply and two fused multiply-adds against
// the correctly rounded reciprocal r = RN(1/s): q0 = RN(x r), e = x - q0 s (exact in an fma),
// v = RN(q0 + e r).  That sequence returns RN(x / s) whenever no intermediate leaves the normal
// range, which `fast` records; otherwise elements take the IEEE division instruction sequence.
struct ScaleCtx {
  float s;    // scale = amax / qmax
  float r;    // RN(1 / s), valid when fast
  bool fast;  // amax within [2^-60, 2^60]
};

__device__ __forceinline__ ScaleCtx make_scale_ctx(float amax, int qmax) {
  ScaleCtx c;
  c.s = __fdiv_rn(amax, (float)qmax);
  c.fast = (amax >= 8.6736174e-19f) && (amax <= 1.1529215e18f);
  c.r = c.fast ? __frcp_rn(c.s) : 0.0f;
  return c;
}

// One element of Fig. 2 after the scale is known: divide_no_nan, round, guard clip.
template <int ROUNDING>
__device__ __forceinline__ int quantize_elem(float x, const ScaleCtx& c, int qmax) {
  float v;
  if (c.fast) {
    float q0 = __fmul_rn(x, c.r);
    float e = __fmaf_rn(-q0, c.s, x);
    v = __fmaf_rn(e, c.r, q0);
  } else {
    v = (c.s == 0.0f) ? 0.0f : __fdiv_rn(x, c.s);
  }
  int q;
  if (ROUNDING == AQT_ROUND_HALF_UP_FLOOR) {
    q = __float2int_rd(__fadd_rn(v, 0.5f));
  } else {
    q = __float2int_rn(v);
  }
  return max(-qmax, min(qmax, q));
}

// Programmatic dependent launch.  Every kernel of the library is launched so that it may start
// while the kernel before it in the stream is still draining, and orders itself with
//   grid_dependency_wait()     returns once the preceding kernel has completed and its memory
//                              operations are visible; placed before the first global-memory access
//                              that could touch anything another kernel reads or writes (set-up
//                              that touches only this CTA's own state runs before it)
//   grid_dependents_launch()   lets the next kernel's CTAs be scheduled once every CTA of this
//                              kernel has executed it (or exited); always after the wait, so that
//                              by the time a later kernel runs, the one before this kernel is complete
// Without the launch attribute both are no-ops.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependents_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

}  // namespace aqt
