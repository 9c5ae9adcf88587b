// Per-tensor amax, scale and FP8 cast of a bf16 tensor (one scale for the whole tensor).
//
// HBM-bound streaming kernels.  CURRENT scaling is two passes (amax, then cast: 2+2+1 B
// per element; the second read comes from L2 when the tensor fits there), GIVEN scaling
// is one pass (2+1 B per element) that still reports the tensor's amax.  Loads are
// 2 x 16 bytes per thread (16 bf16), stores 16 bytes (16 codes).  amax is the integer
// maximum of the sign-stripped bf16 bit patterns (exact, order-independent; NaN
// patterns are skipped), reduced by shuffles and one atomicMax per CTA.
//
// Two launch forms.  Without a workspace: a reset kernel, the amax kernel and the cast kernel.
// With a workspace: two kernels for up to TWEO_MAX_QUANT_BATCH tensors at once -- one reduces
// every tensor's amax into the workspace, the other casts every tensor with the scale derived
// from it, and its last CTA writes the scalars out and leaves the workspace zeroed for the
// next call (so no reset kernel).  A linear layer's three casts (X, W, dY) then cost two
// launches instead of nine, which matters because the tensors of a transformer block are
// small enough for launch cost to rival streaming time.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "common.cuh"

namespace tweo_detail {
tweo_status_t launch_amax_prologue(const uint16_t* x, int64_t n, float* amax, uint32_t* sat_count, const float* scale_in,
                                   float* scale_inv, cudaStream_t st);
}

namespace {

using namespace tweo_detail;

constexpr int kThreads = 256;

// m: this thread's maximum as a bf16 bit pattern
__device__ __forceinline__ void cta_amax_to_global(uint32_t m, float* amax) {
  __shared__ uint32_t part[kThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) m = max(m, part[w]);
    // non-negative binary32 values order like their bit patterns
    if (m) atomicMax(reinterpret_cast<unsigned int*>(amax), m << 16);
  }
}

// The single-tensor kernels are launched in a chain too (see chain_wait() in common.cuh): the launch latency and
// the few instructions before the wait overlap the tail of the kernel before them.
__global__ void init_kernel(float* amax, uint32_t* sat_count, const float* scale_in, float* scale_inv) {
  chain_release();
  chain_wait();
  *amax = 0.0f;
  if (sat_count) *sat_count = 0u;
  if (scale_in) *scale_inv = __fdiv_rn(1.0f, *scale_in);
}

__global__ void __launch_bounds__(kThreads) amax_kernel(const uint16_t* x, int64_t n, float* amax) {
  chain_release();
  chain_wait();
  const int64_t nvec = n >> 3;
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  const int64_t stride = (int64_t)gridDim.x * kThreads * 4;
  uint32_t m = 0;
  for (int64_t base = (int64_t)blockIdx.x * kThreads * 4 + threadIdx.x; base < nvec; base += stride) {
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      int64_t i = base + (int64_t)u * kThreads;
      v[u] = i < nvec ? __ldg(xv + i) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      m = absmax_bits(m, v[u].x);
      m = absmax_bits(m, v[u].y);
      m = absmax_bits(m, v[u].z);
      m = absmax_bits(m, v[u].w);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < 8) {
    int64_t i = (nvec << 3) + threadIdx.x;
    if (i < n) m = absmax_bits(m, (uint32_t)x[i]);
  }
  cta_amax_to_global(absmax_fold(m), amax);
}

// 16 elements: two 16-byte loads -> one 16-byte store.  SAT counts elements whose scaled value
// exceeds the format's range, AMAX folds |x| into the running maximum m2.  NaN inputs come out of the
// converter as the code 0x7F (see cvt_fp8x2).
template <int FMT, bool SAT, bool AMAX>
__device__ __forceinline__ uint4 cast16(const uint4 a, const uint4 b, float scale, uint32_t& sat, float& m0, float& m1) {
  const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
  uint32_t c[8];
  const float fmax = FMT == TWEO_E4M3 ? kE4M3Max : kE5M2Max;
  const uint64_t ss = pack_f32x2(scale, scale);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float lo, hi;
    unpack_f32x2(mul_f32x2(bf16x2_to_f32x2(w[j]), ss), lo, hi);   // one packed multiply, each lane rounded once
    if (SAT) sat += (fabsf(lo) > fmax) + (fabsf(hi) > fmax);
    c[j] = cvt_fp8x2<FMT>(lo, hi);
    if (AMAX) absmax_f32(m0, m1, w[j]);
  }
  return make_uint4(c[0] | (c[1] << 16), c[2] | (c[3] << 16), c[4] | (c[5] << 16), c[6] | (c[7] << 16));
}

// CURRENT mode reads *amax (finished by the previous kernel) and derives the scale;
// GIVEN mode reads *scale and accumulates amax while casting.
// U: pairs of 16-byte loads in flight per thread (the deeper variant for large tensors, as in the batched form).
template <int FMT, bool GIVEN, bool SAT, int U>
__global__ void __launch_bounds__(kThreads)
cast_kernel(const uint16_t* x, int64_t n, float* scale, float* scale_inv, float* amax, uint8_t* q,
            uint32_t* sat_count) {
  chain_release();
  chain_wait();
  float s;
  if (GIVEN) {
    s = *scale;
  } else {
    s = scale_from_amax(*amax, FMT);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      *scale = s;
      *scale_inv = __fdiv_rn(1.0f, s);
    }
  }
  const int64_t n16 = n >> 4;
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  uint4* qv = reinterpret_cast<uint4*>(q);
  const int64_t stride = (int64_t)gridDim.x * kThreads * U;
  uint32_t sat = 0;
  float m0 = 0.0f, m1 = 0.0f;   // running maximum of |x| (GIVEN mode), two lanes; fmaxf skips NaN
  for (int64_t base = (int64_t)blockIdx.x * kThreads * U + threadIdx.x; base < n16; base += stride) {
    uint4 v[U][2];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      int64_t i = base + (int64_t)u * kThreads;
      if (i < n16) {
        v[u][0] = __ldcs(xv + 2 * i);
        v[u][1] = __ldcs(xv + 2 * i + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      int64_t i = base + (int64_t)u * kThreads;
      if (i < n16) __stcs(qv + i, cast16<FMT, SAT, GIVEN>(v[u][0], v[u][1], s, sat, m0, m1));
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < 16) {  // ragged tail: n % 16 elements
    int64_t i = (n16 << 4) + threadIdx.x;
    if (i < n) {
      uint32_t w = x[i];
      float v = __fmul_rn(bf16lo_to_f32(w), s);
      sat += fabsf(v) > (FMT == TWEO_E4M3 ? kE4M3Max : kE5M2Max);
      q[i] = (uint8_t)(cvt_fp8x2<FMT>(v, 0.0f) & 0xFFu);
      if (GIVEN) absmax_f32(m0, m1, w);
    }
  }
  if (SAT) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sat += __shfl_xor_sync(0xFFFFFFFFu, sat, o);
    if ((threadIdx.x & 31) == 0 && sat) atomicAdd(sat_count, sat);
  }
  if (GIVEN) cta_amax_to_global(absmax_f32_bits(m0, m1), amax);
}

// ---------------------------------------------------------------------------------------
// Batched form with a workspace (CURRENT scaling): no reset kernel and no atomics.
//   kernel 1: every CTA writes the maximum of its share of each tensor to its own workspace
//             slot (so the workspace needs no particular contents on entry);
//   kernel 2 (one launch per FP8 format present): every CTA first reduces the slots of a
//             tensor to its amax (a few KB from L2), derives the scale and casts its share;
//             CTA 0 writes amax, scale and scale_inv.
struct QTensor {
  const uint16_t* x;
  uint8_t* q;
  int64_t n;
  float* scale;
  float* scale_inv;
  float* amax;
  int32_t fmt;
  int32_t pad;
};
struct QBatch {
  QTensor t[TWEO_MAX_QUANT_BATCH];
  int32_t count;
  int32_t amax_grid;  // CTAs of kernel 1 = slots per tensor
};
constexpr int kMaxAmaxGrid = 2048;  // slots per tensor in the workspace

__device__ __forceinline__ uint32_t cta_max(uint32_t m, uint32_t* part) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __syncthreads();  // part[] may still be read from the previous use
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
  __syncthreads();
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) m = max(m, part[w]);
  return m;
}

// U: 16-byte loads in flight per thread.  Large batches take the deeper variant (more bytes in flight per SM);
// small ones the shallow one, whose smaller per-CTA share keeps all SMs busy to the end.
template <int U>
__global__ void __launch_bounds__(kThreads) amax_batch_kernel(const __grid_constant__ QBatch b, uint32_t* slots) {
  __shared__ uint32_t part[kThreads / 32];
  chain_release();
  chain_wait();
#pragma unroll 1
  for (int ti = 0; ti < b.count; ++ti) {
    const int64_t n = b.t[ti].n;
    const int64_t nvec = n >> 3;
    const uint16_t* x = b.t[ti].x;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    const int64_t stride = (int64_t)gridDim.x * kThreads * U;
    float m0 = 0.0f, m1 = 0.0f;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * U + threadIdx.x; base < nvec; base += stride) {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        int64_t i = base + (int64_t)u * kThreads;
        v[u] = i < nvec ? __ldg(xv + i) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        absmax_f32(m0, m1, v[u].x);
        absmax_f32(m0, m1, v[u].y);
        absmax_f32(m0, m1, v[u].z);
        absmax_f32(m0, m1, v[u].w);
      }
    }
    if (blockIdx.x == 0 && threadIdx.x < 8) {
      int64_t i = (nvec << 3) + threadIdx.x;
      if (i < n) absmax_f32(m0, m1, (uint32_t)x[i]);
    }
    const uint32_t m = cta_max(absmax_f32_bits(m0, m1), part);
    if (threadIdx.x == 0) slots[ti * kMaxAmaxGrid + blockIdx.x] = m;
  }
}

// U: pairs of 16-byte loads in flight per thread (see amax_batch_kernel)
template <int FMT, int U>
__global__ void __launch_bounds__(kThreads) cast_batch_kernel(const __grid_constant__ QBatch b, const uint32_t* slots) {
  __shared__ uint32_t part[kThreads / 32];
  chain_release();
  chain_wait();
#pragma unroll 1
  for (int ti = 0; ti < b.count; ++ti) {
    if (b.t[ti].fmt != FMT) continue;
    uint32_t m = 0;
    for (int k = threadIdx.x; k < b.amax_grid; k += kThreads) m = max(m, __ldcg(slots + ti * kMaxAmaxGrid + k));
    m = cta_max(m, part);
    const float amax = __uint_as_float(m << 16);  // non-negative bf16 pattern -> binary32
    const float s = scale_from_amax(amax, FMT);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      *b.t[ti].amax = amax;
      *b.t[ti].scale = s;
      *b.t[ti].scale_inv = __fdiv_rn(1.0f, s);
    }
    const int64_t n = b.t[ti].n;
    const int64_t n16 = n >> 4;
    const uint16_t* x = b.t[ti].x;
    uint8_t* q = b.t[ti].q;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    uint4* qv = reinterpret_cast<uint4*>(q);
    const int64_t stride = (int64_t)gridDim.x * kThreads * U;
    uint32_t sat = 0;
    float mm0 = 0.0f, mm1 = 0.0f;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * U + threadIdx.x; base < n16; base += stride) {
      uint4 v[U][2];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        int64_t i = base + (int64_t)u * kThreads;
        if (i < n16) {
          v[u][0] = __ldcs(xv + 2 * i);
          v[u][1] = __ldcs(xv + 2 * i + 1);
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        int64_t i = base + (int64_t)u * kThreads;
        if (i < n16) __stcs(qv + i, cast16<FMT, false, false>(v[u][0], v[u][1], s, sat, mm0, mm1));
      }
    }
    if (blockIdx.x == 0 && threadIdx.x < 16) {  // ragged tail: n % 16 elements
      int64_t i = (n16 << 4) + threadIdx.x;
      if (i < n) {
        float v = __fmul_rn(bf16lo_to_f32((uint32_t)x[i]), s);
        q[i] = (uint8_t)(cvt_fp8x2<FMT>(v, 0.0f) & 0xFFu);
      }
    }
  }
}

// Batched form for GIVEN (delayed / static) scales: one reset kernel for all tensors of the batch, then one
// single-pass cast kernel per FP8 format present; every CTA folds its share of a tensor into that tensor's amax
// with one atomicMax.  Three launches for a linear's (or two linears') tensors instead of two per tensor.
__global__ void init_batch_kernel(const __grid_constant__ QBatch b) {
  chain_release();
  chain_wait();
  const int ti = threadIdx.x;
  if (ti < b.count) {
    *b.t[ti].amax = 0.0f;
    *b.t[ti].scale_inv = __fdiv_rn(1.0f, *b.t[ti].scale);
  }
}

template <int FMT, int U>
__global__ void __launch_bounds__(kThreads) cast_given_batch_kernel(const __grid_constant__ QBatch b) {
  chain_release();
  chain_wait();
#pragma unroll 1
  for (int ti = 0; ti < b.count; ++ti) {
    if (b.t[ti].fmt != FMT) continue;
    const float s = *b.t[ti].scale;
    const int64_t n = b.t[ti].n;
    const int64_t n16 = n >> 4;
    const uint16_t* x = b.t[ti].x;
    uint8_t* q = b.t[ti].q;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    uint4* qv = reinterpret_cast<uint4*>(q);
    const int64_t stride = (int64_t)gridDim.x * kThreads * U;
    uint32_t sat = 0;
    float m0 = 0.0f, m1 = 0.0f;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * U + threadIdx.x; base < n16; base += stride) {
      uint4 v[U][2];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        int64_t i = base + (int64_t)u * kThreads;
        if (i < n16) {
          v[u][0] = __ldcs(xv + 2 * i);
          v[u][1] = __ldcs(xv + 2 * i + 1);
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        int64_t i = base + (int64_t)u * kThreads;
        if (i < n16) __stcs(qv + i, cast16<FMT, false, true>(v[u][0], v[u][1], s, sat, m0, m1));
      }
    }
    if (blockIdx.x == 0 && threadIdx.x < 16) {  // ragged tail: n % 16 elements
      int64_t i = (n16 << 4) + threadIdx.x;
      if (i < n) {
        const uint32_t w = x[i];
        q[i] = (uint8_t)(cvt_fp8x2<FMT>(__fmul_rn(bf16lo_to_f32(w), s), 0.0f) & 0xFFu);
        absmax_f32(m0, m1, w);
      }
    }
    __syncthreads();  // the reduction's shared array may still be read from the previous tensor
    cta_amax_to_global(absmax_f32_bits(m0, m1), b.t[ti].amax);
  }
}

int grid_for(int64_t work_items, int per_cta, int ctas_per_sm);

// Launches the batched form for descs[idx[0..count)] (all CURRENT scaling, no saturation count).
tweo_status_t launch_batch(const tweo_quant_desc_t* descs, const int* idx, int count, void* ws, cudaStream_t st) {
  QBatch b;
  b.count = count;
  int64_t vec8 = 0, vec16[2] = {0, 0};
  for (int i = 0; i < count; ++i) {
    const tweo_quant_desc_t& d = descs[idx[i]];
    b.t[i] = QTensor{d.x, d.q, d.n, d.scale, d.scale_inv, d.amax, d.fmt, 0};
    vec8 += d.n >> 3;
    vec16[d.fmt] += d.n >> 4;
  }
  // the deeper variants once a launch has at least two full sweeps of the capped grid at their depth
  const int64_t sweep = (int64_t)sm_count() * 8 * kThreads;
  const bool deep_amax = vec8 >= 2 * sweep * 8;
  b.amax_grid = grid_for(vec8, kThreads * (deep_amax ? 8 : 4), 8);
  if (b.amax_grid > kMaxAmaxGrid) b.amax_grid = kMaxAmaxGrid;
  uint32_t* slots = reinterpret_cast<uint32_t*>(ws);
  if (deep_amax) TWEO_CUDA_TRY(launch_chain(amax_batch_kernel<8>, dim3(b.amax_grid), dim3(kThreads), 0, st, 0, b, slots));
  else TWEO_CUDA_TRY(launch_chain(amax_batch_kernel<4>, dim3(b.amax_grid), dim3(kThreads), 0, st, 0, b, slots));
  count_launch();
  bool has[2] = {false, false};
  for (int i = 0; i < count; ++i) has[b.t[i].fmt] = true;
  if (has[TWEO_E4M3]) {
    if (vec16[TWEO_E4M3] >= 2 * sweep * 4)
      TWEO_CUDA_TRY(launch_chain(cast_batch_kernel<TWEO_E4M3, 4>, dim3(grid_for(vec16[TWEO_E4M3], kThreads * 4, 8)), dim3(kThreads), 0, st, 0, b,
                                 (const uint32_t*)slots));
    else
      TWEO_CUDA_TRY(launch_chain(cast_batch_kernel<TWEO_E4M3, 2>, dim3(grid_for(vec16[TWEO_E4M3], kThreads * 2, 8)), dim3(kThreads), 0, st, 0, b,
                                 (const uint32_t*)slots));
    count_launch();
  }
  if (has[TWEO_E5M2]) {
    if (vec16[TWEO_E5M2] >= 2 * sweep * 4)
      TWEO_CUDA_TRY(launch_chain(cast_batch_kernel<TWEO_E5M2, 4>, dim3(grid_for(vec16[TWEO_E5M2], kThreads * 4, 8)), dim3(kThreads), 0, st, 0, b,
                                 (const uint32_t*)slots));
    else
      TWEO_CUDA_TRY(launch_chain(cast_batch_kernel<TWEO_E5M2, 2>, dim3(grid_for(vec16[TWEO_E5M2], kThreads * 2, 8)), dim3(kThreads), 0, st, 0, b,
                                 (const uint32_t*)slots));
    count_launch();
  }
  return check_launch("quantize batch kernels");
}

// Launches the given-scale batched form for descs[idx[0..count)] (no saturation count).
tweo_status_t launch_given_batch(const tweo_quant_desc_t* descs, const int* idx, int count, cudaStream_t st) {
  QBatch b;
  b.count = count;
  b.amax_grid = 0;
  int64_t vec16[2] = {0, 0};
  for (int i = 0; i < count; ++i) {
    const tweo_quant_desc_t& d = descs[idx[i]];
    b.t[i] = QTensor{d.x, d.q, d.n, d.scale, d.scale_inv, d.amax, d.fmt, 0};
    vec16[d.fmt] += d.n >> 4;
  }
  TWEO_CUDA_TRY(launch_chain(init_batch_kernel, dim3(1), dim3(32), 0, st, 0, b));
  count_launch();
  const int64_t sweep = (int64_t)sm_count() * 8 * kThreads;
  bool has[2] = {false, false};
  for (int i = 0; i < count; ++i) has[b.t[i].fmt] = true;
  if (has[TWEO_E4M3]) {
    if (vec16[TWEO_E4M3] >= 2 * sweep * 4)
      TWEO_CUDA_TRY(launch_chain(cast_given_batch_kernel<TWEO_E4M3, 4>, dim3(grid_for(vec16[TWEO_E4M3], kThreads * 4, 8)),
                                 dim3(kThreads), 0, st, 0, b));
    else
      TWEO_CUDA_TRY(launch_chain(cast_given_batch_kernel<TWEO_E4M3, 2>, dim3(grid_for(vec16[TWEO_E4M3], kThreads * 2, 8)),
                                 dim3(kThreads), 0, st, 0, b));
    count_launch();
  }
  if (has[TWEO_E5M2]) {
    if (vec16[TWEO_E5M2] >= 2 * sweep * 4)
      TWEO_CUDA_TRY(launch_chain(cast_given_batch_kernel<TWEO_E5M2, 4>, dim3(grid_for(vec16[TWEO_E5M2], kThreads * 4, 8)),
                                 dim3(kThreads), 0, st, 0, b));
    else
      TWEO_CUDA_TRY(launch_chain(cast_given_batch_kernel<TWEO_E5M2, 2>, dim3(grid_for(vec16[TWEO_E5M2], kThreads * 2, 8)),
                                 dim3(kThreads), 0, st, 0, b));
    count_launch();
  }
  return check_launch("quantize given-scale batch kernels");
}

constexpr size_t kBatchWsBytes = (size_t)TWEO_MAX_QUANT_BATCH * kMaxAmaxGrid * sizeof(uint32_t);  // 64 KB

int grid_for(int64_t work_items, int per_cta, int ctas_per_sm) {
  return balanced_grid((work_items + per_cta - 1) / per_cta, (int64_t)sm_count() * ctas_per_sm);
}

tweo_status_t check_desc(const tweo_quant_desc_t& d) {
  if (d.n < 0 || !d.scale || !d.scale_inv || !d.amax) return TWEO_ERR_INVALID_ARG;
  if (d.n > 0 && (!d.x || !d.q)) return TWEO_ERR_INVALID_ARG;
  if (d.fmt != TWEO_E4M3 && d.fmt != TWEO_E5M2) return TWEO_ERR_INVALID_ARG;
  if (d.mode != TWEO_SCALE_CURRENT && d.mode != TWEO_SCALE_GIVEN) return TWEO_ERR_INVALID_ARG;
  if (!aligned16(d.x) || !aligned16(d.q)) return TWEO_ERR_ALIGNMENT;
  return TWEO_OK;
}

// One tensor as separate kernels: reset, amax (CURRENT only), cast.
template <int FMT, bool GIVEN, bool SAT>
cudaError_t launch_cast(const tweo_quant_desc_t& d, cudaStream_t st) {
  const int64_t n16 = d.n >> 4;
  const int64_t sweep = (int64_t)sm_count() * 8 * kThreads;
  if (n16 >= 2 * sweep * 4)
    return launch_chain(cast_kernel<FMT, GIVEN, SAT, 4>, dim3(grid_for(n16, kThreads * 4, 8)), dim3(kThreads), 0, st, 0,
                        d.x, d.n, d.scale, d.scale_inv, d.amax, d.q, d.sat_count);
  return launch_chain(cast_kernel<FMT, GIVEN, SAT, 2>, dim3(grid_for(n16, kThreads * 2, 8)), dim3(kThreads), 0, st, 0, d.x,
                      d.n, d.scale, d.scale_inv, d.amax, d.q, d.sat_count);
}

tweo_status_t launch_single(const tweo_quant_desc_t& d, cudaStream_t st) {
  const bool given = d.mode == TWEO_SCALE_GIVEN;
  tweo_status_t ps = tweo_detail::launch_amax_prologue(d.x, d.n, d.amax, d.sat_count,
                                                       given ? (const float*)d.scale : (const float*)nullptr, d.scale_inv, st);
  if (ps != TWEO_OK) return ps;
  const bool sat = d.sat_count != nullptr;
  cudaError_t e;
  if (d.fmt == TWEO_E4M3) {
    if (given) e = sat ? launch_cast<TWEO_E4M3, true, true>(d, st) : launch_cast<TWEO_E4M3, true, false>(d, st);
    else e = sat ? launch_cast<TWEO_E4M3, false, true>(d, st) : launch_cast<TWEO_E4M3, false, false>(d, st);
  } else {
    if (given) e = sat ? launch_cast<TWEO_E5M2, true, true>(d, st) : launch_cast<TWEO_E5M2, true, false>(d, st);
    else e = sat ? launch_cast<TWEO_E5M2, false, true>(d, st) : launch_cast<TWEO_E5M2, false, false>(d, st);
  }
  TWEO_CUDA_TRY(e);
  count_launch();
  return check_launch("tweo_quantize_per_tensor");
}

// Tensors with CURRENT scaling and no saturation count go through the batched kernels when a
// workspace is there; two or more GIVEN-scale tensors without saturation count share the given-scale
// batch kernels; the others are launched one by one.
tweo_status_t quantize_many(const tweo_quant_desc_t* descs, int count, void* ws, size_t ws_bytes, cudaStream_t st) {
  for (int i = 0; i < count; ++i) {
    tweo_status_t s = check_desc(descs[i]);
    if (s != TWEO_OK) return s;
  }
  const bool have_ws = ws && ws_bytes >= kBatchWsBytes && aligned16(ws);
  int idx[TWEO_MAX_QUANT_BATCH], idxg[TWEO_MAX_QUANT_BATCH];
  int nb = 0, ng = 0;
  for (int i = 0; i < count; ++i) {
    if (have_ws && descs[i].mode == TWEO_SCALE_CURRENT && !descs[i].sat_count) idx[nb++] = i;
    else if (count > 1 && descs[i].mode == TWEO_SCALE_GIVEN && !descs[i].sat_count) idxg[ng++] = i;
    else {
      tweo_status_t s = launch_single(descs[i], st);
      if (s != TWEO_OK) return s;
    }
  }
  if (ng == 1) {   // a lone given-scale tensor gains nothing from the batched form
    tweo_status_t s = launch_single(descs[idxg[0]], st);
    if (s != TWEO_OK) return s;
  } else if (ng > 1) {
    tweo_status_t s = launch_given_batch(descs, idxg, ng, st);
    if (s != TWEO_OK) return s;
  }
  if (nb > 0) return launch_batch(descs, idx, nb, ws, st);
  return TWEO_OK;
}

}  // namespace

namespace tweo_detail {
// The first launches of every one-tensor cast (FP8 here, FP4 in fp4.cu): the reset of amax (and of the saturation
// counter; with a given scale also its reciprocal), then, for current scaling (scale_in == nullptr), the amax pass.
tweo_status_t launch_amax_prologue(const uint16_t* x, int64_t n, float* amax, uint32_t* sat_count, const float* scale_in,
                                   float* scale_inv, cudaStream_t st) {
  TWEO_CUDA_TRY(launch_chain(init_kernel, dim3(1), dim3(1), 0, st, 0, amax, sat_count, scale_in, scale_inv));
  count_launch();
  if (!scale_in) {
    TWEO_CUDA_TRY(launch_chain(amax_kernel, dim3(grid_for(n >> 3, kThreads * 4, 8)), dim3(kThreads), 0, st, 0, x, n, amax));
    count_launch();
  }
  return TWEO_OK;
}

size_t quantize_workspace_bytes() { return kBatchWsBytes; }
}

extern "C" tweo_status_t tweo_quantize_per_tensor(const uint16_t* x, int64_t n, int32_t fmt, int32_t mode,
                                                  float* scale, float* scale_inv, float* amax, uint8_t* q,
                                                  uint32_t* sat_count, void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_quantize_per_tensor " "x=%p n=%lld fmt=%d mode=%d q=%p ws=%p", (const void*)x, (long long)n, fmt, mode, (void*)q, ws);
  tweo_quant_desc_t d{x, n, fmt, mode, scale, scale_inv, amax, q, sat_count};
  return quantize_many(&d, 1, ws, ws_bytes, (cudaStream_t)stream);
}

extern "C" tweo_status_t tweo_quantize_per_tensor_batch(const tweo_quant_desc_t* descs, int32_t count, void* ws,
                                                        size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_quantize_per_tensor_batch " "descs=%p count=%d ws=%p ws_bytes=%zu", (const void*)descs, count, ws, ws_bytes);
  if (!descs || count < 1 || count > TWEO_MAX_QUANT_BATCH) return TWEO_ERR_INVALID_ARG;
  if (ws && !aligned16(ws)) return TWEO_ERR_ALIGNMENT;
  return quantize_many(descs, count, ws, ws_bytes, (cudaStream_t)stream);
}
