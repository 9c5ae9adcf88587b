// Shared host/device helpers of the CUDA library (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "tweo.h"

namespace tweo_detail {

// Number of SMs the persistent kernels size their grids for (queried once per device).
int sm_count();

// Book-keeping shared by all translation units.
void count_launch(int n = 1);
tweo_status_t cuda_fail(cudaError_t e, const char* what);  // records text, returns TWEO_ERR_CUDA
tweo_status_t check_launch(const char* what);              // cudaGetLastError after a launch

// TWEO_LOG=1 in the environment (read once): every entry point prints its name and its scalar arguments to stderr
// before it does anything else -- shapes, formats, pitches, which optional pointers are set.  Nothing is read from
// the device and nothing is synchronised.
bool log_enabled();
void log_call(const char* fmt, ...) __attribute__((format(printf, 1, 2)));

// Device status word (bounded waits that expired); lives with the GEMM kernels.
tweo_status_t read_and_clear_device_status(cudaStream_t stream);
unsigned int* device_status_word();  // its device address on the current device (nullptr on failure)

// Grid of a streaming kernel whose CTAs walk `iters` equal pieces of work with a grid-stride loop, at most `cap`
// CTAs: every CTA gets the same number of pieces (or one less), so no SM waits for a straggler that drew one more
// sweep than the average -- with iters = 3.5 x cap a capped grid would finish at 4 sweeps, 13 % late.
inline int balanced_grid(int64_t iters, int64_t cap) {
  if (cap < 1) cap = 1;
  if (iters <= cap) return (int)(iters < 1 ? 1 : iters);
  const int64_t per = (iters + cap - 1) / cap;
  return (int)((iters + per - 1) / per);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// One-time set-up that CUDA keeps per device (function attributes): `mask` has one bit per device.
// device_once_pending() is true while the current device still needs it; two host threads that race
// here both run the (idempotent) set-up.  Devices beyond 63 are set up on every call.
inline bool device_once_pending(std::atomic<uint64_t>& mask, int* dev) {
  *dev = -1;
  if (cudaGetDevice(dev) != cudaSuccess || *dev < 0 || *dev >= 64) return true;
  return (mask.load(std::memory_order_acquire) & (1ull << *dev)) == 0;
}
inline void device_once_done(std::atomic<uint64_t>& mask, int dev) {
  if (dev >= 0 && dev < 64) mask.fetch_or(1ull << dev, std::memory_order_release);
}

}  // namespace tweo_detail

#define TWEO_LOG_CALL(...)                                               \
  do {                                                                   \
    if (tweo_detail::log_enabled()) tweo_detail::log_call(__VA_ARGS__);  \
  } while (0)

#define TWEO_CUDA_TRY(expr)                                              \
  do {                                                                   \
    cudaError_t _e = (expr);                                             \
    if (_e != cudaSuccess) return tweo_detail::cuda_fail(_e, #expr);     \
  } while (0)

#ifdef __CUDACC__
namespace tweo_detail {

// Launches `kern` with `cluster` CTAs per cluster (0: none) as a programmatic dependent of the kernel before it
// on the stream (see chain_wait()).
template <typename... KArgs, typename... Args>
cudaError_t launch_chain(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, unsigned cluster,
                         Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (cluster > 0) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

constexpr float kE4M3Max = 448.0f;
constexpr float kE5M2Max = 57344.0f;

__device__ __forceinline__ float fp8_max(int fmt) { return fmt == TWEO_E4M3 ? kE4M3Max : kE5M2Max; }

// Two binary32 values -> two FP8 codes (round-to-nearest-even, saturating to the
// largest finite value); `lo` lands in bits 0-7, `hi` in bits 8-15.  A NaN input gives the
// code 0x7F in both formats whatever its sign or payload, +-inf the largest finite code: that
// is what the converter returns (checked for quiet, signalling, positive and negative NaNs, and
// by the all-bf16-patterns parity test), so no fix-up instructions are spent on it.
template <int FMT>
__device__ __forceinline__ uint32_t cvt_fp8x2(float lo, float hi) {
  uint16_t r;
  if (FMT == TWEO_E4M3)
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  else
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// binary32 -> bf16 bits, round-to-nearest-even.
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(f));
  return r;
}
// packs bf16(lo) | bf16(hi) << 16
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Packed binary32 pairs (sm_100: one instruction works on two IEEE lanes, each rounded to nearest-even exactly as
// the scalar instruction would).  A pair lives in a 64-bit register; packing and unpacking are register moves.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
// the two bf16 values of a packed word as a binary32 pair (exact)
__device__ __forceinline__ uint64_t bf16x2_to_f32x2(uint32_t w) { return pack_f32x2(bf16lo_to_f32(w), bf16hi_to_f32(w)); }
__device__ __forceinline__ uint32_t f32x2_pair_to_bf16x2(uint64_t v) {
  float lo, hi;
  unpack_f32x2(v, lo, hi);
  return f32x2_to_bf16x2(lo, hi);
}

// per-tensor scale from amax: fl32(FP8MAX / amax); 1 for amax == 0 or non-finite;
// clamped to FLT_MAX when the quotient overflows.
__device__ __forceinline__ float scale_from_amax(float amax, int fmt) {
  float s = 1.0f;
  if (amax > 0.0f && amax < __int_as_float(0x7F800000)) {
    s = __fdiv_rn(fp8_max(fmt), amax);
    if (s > 3.402823466e38f) s = 3.402823466e38f;
  }
  return s;
}

// Running maximum of |x| over packed pairs of bf16, kept as two 16-bit lanes of sign-stripped bit
// patterns (which order like the magnitudes); NaN patterns (> 0x7F80) count as 0.  Four integer
// SIMD instructions per pair of elements.
__device__ __forceinline__ uint32_t absmax_bits(uint32_t m2, uint32_t w) {
  uint32_t a = w & 0x7FFF7FFFu;
  a &= __vcmpleu2(a, 0x7F807F80u);
  return __vmaxu2(m2, a);
}
// The same running maximum kept as two binary32 values (fmaxf skips NaN by itself): four plain instructions per
// pair of elements.  absmax_f32_bits() gives the result as a bf16 bit pattern like absmax_fold().
__device__ __forceinline__ void absmax_f32(float& m0, float& m1, uint32_t w) {
  m0 = fmaxf(m0, fabsf(bf16lo_to_f32(w)));
  m1 = fmaxf(m1, fabsf(bf16hi_to_f32(w)));
}
__device__ __forceinline__ uint32_t absmax_f32_bits(float m0, float m1) { return __float_as_uint(fmaxf(m0, m1)) >> 16; }
// the larger of the two lanes: the bit pattern of max |x| as a bf16 value
__device__ __forceinline__ uint32_t absmax_fold(uint32_t m2) { return max(m2 & 0xFFFFu, m2 >> 16); }
// Programmatic dependent launch: a kernel launched with launch_chain() may become resident while the kernel
// before it on the stream is still running (its launch latency and prologue are hidden); it must not touch
// global memory before chain_wait(), which returns once that kernel has completed and its writes are visible.
// chain_release() lets the next kernel of the chain start launching.  Both are no-ops in a kernel that was
// launched the ordinary way.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

}  // namespace tweo_detail
#endif  // __CUDACC__
