// TWEO penalty (Eq. 3) and its gradient in one streaming pass over each block output.
//
// HBM-bound: 2 B read + 2 B (bf16 grad) or 4 B (fp32 grad) written per element, ~8 flop.
// One launch covers all L block outputs: grid = (blocks per tensor, L).  Each thread
// streams 16-byte vectors (8 bf16) with four independent loads in flight, accumulates
// sum |a|^p per vector in binary32 and across vectors in binary64, the CTA reduces with
// shuffles and writes ONE partial sum to the scratch memory.  A second, one-CTA kernel
// (launched in the same chain, so its launch and set-up overlap the first) adds the
// partials in a fixed order and writes the losses: the result does not depend on
// scheduling, and the streaming CTAs end without a fence, a ticket or a wait -- a
// last-CTA-reduces scheme cost 3.4 us at the end of every call (fence, atomic, a dependent
// round trip to L2 behind the slowest CTA), a third of the pass over a [8192 x 768] tensor.
#include <cuda_bf16.h>

#include <mutex>

#include "common.cuh"

namespace tweo_detail {

constexpr int kLossThreads = 256;
constexpr int kLossUnroll = 4;  // 16-byte vectors in flight per thread
// CTAs per SM the grid is sized for.  Not the most that fit: in a launch chain the CTAs of the NEXT kernel should
// find room on the SMs while this kernel still runs, so that they sit at their dependency wait when it ends
// (measured on [16384 x 2048]: 6 per SM 28.0 us, 4 per SM 25.6 us per call; 3 and 5 in between).
constexpr int kLossCtasPerSm = 4;

int loss_blocks_per_tensor(int64_t n, int L) {
  if (L < 1) L = 1;
  int64_t vec = n / 8;
  int64_t want = (vec + (int64_t)kLossThreads * kLossUnroll - 1) / ((int64_t)kLossThreads * kLossUnroll);
  int64_t cap = ((int64_t)sm_count() * kLossCtasPerSm + L - 1) / L;  // one wave of resident CTAs overall
  return balanced_grid(want, cap);
}

}  // namespace tweo_detail

namespace {

using namespace tweo_detail;

struct LossPtrs {
  const uint16_t* a[TWEO_MAX_BLOCKS];
  void* g[TWEO_MAX_BLOCKS];
};

struct LossArgs {
  int64_t n;        // elements per tensor
  int L;
  float p;
  float k_grad;     // fl32( grad_coeff * p / (n * (tau+eps)^p) ), rounded once on the host
  double inv_norm;  // 1 / (n * (tau+eps)^p)
  float* loss;
  float* loss_per_block;  // or nullptr
  double* partials;       // [L][gridDim.x]
  int parts_per_tensor;   // gridDim.x of the streaming kernel
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
  return v;
}

// One 16-byte vector (8 bf16).  p = 4: packed binary32 pairs -- s = a*a is exact (8-bit significands), a^3 = s*a
// too (24 bits), so g = fl32(k * a^3) rounds once; the a^4 terms are folded into the running pair `acc2` by a
// fused multiply-add (acc2 += s*s), which the caller empties into its binary64 sum once per loop iteration.
// Other p: binary64 pow (keeps the 1e-5 budget for any p > 1), terms added to `vsum`.
template <bool FAST, bool GRAD, bool GRAD_F32>
__device__ __forceinline__ void process_vec(const uint4 v, float k, float p, uint64_t& acc2, float& vsum,
                                            uint4* gout_bf16, float4* gout_f32) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  if (FAST) {
    const uint64_t kk = pack_f32x2(k, k);
    uint64_t g2[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t a2 = bf16x2_to_f32x2(w[j]);
      const uint64_t s2 = mul_f32x2(a2, a2);
      acc2 = fma_f32x2(s2, s2, acc2);
      if (GRAD) g2[j] = mul_f32x2(kk, mul_f32x2(s2, a2));
    }
    if (GRAD) {
      if (GRAD_F32) {
        float g[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) unpack_f32x2(g2[j], g[2 * j], g[2 * j + 1]);
        gout_f32[0] = make_float4(g[0], g[1], g[2], g[3]);
        gout_f32[1] = make_float4(g[4], g[5], g[6], g[7]);
      } else {
        *gout_bf16 = make_uint4(f32x2_pair_to_bf16x2(g2[0]), f32x2_pair_to_bf16x2(g2[1]), f32x2_pair_to_bf16x2(g2[2]),
                                f32x2_pair_to_bf16x2(g2[3]));
      }
    }
  } else {
  float g[8];
  float t[8];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float a0 = bf16lo_to_f32(w[j]), a1 = bf16hi_to_f32(w[j]);
    double m0 = fabs((double)a0), m1 = fabs((double)a1);
    t[2 * j] = (float)pow(m0, (double)p);
    t[2 * j + 1] = (float)pow(m1, (double)p);
    if (GRAD) {
      g[2 * j] = a0 == 0.0f ? 0.0f : (float)((double)k * copysign(pow(m0, (double)p - 1.0), (double)a0));
      g[2 * j + 1] = a1 == 0.0f ? 0.0f : (float)((double)k * copysign(pow(m1, (double)p - 1.0), (double)a1));
    }
  }
  vsum += ((t[0] + t[1]) + (t[2] + t[3])) + ((t[4] + t[5]) + (t[6] + t[7]));
  if (GRAD) {
    if (GRAD_F32) {
      gout_f32[0] = make_float4(g[0], g[1], g[2], g[3]);
      gout_f32[1] = make_float4(g[4], g[5], g[6], g[7]);
    } else {
      *gout_bf16 = make_uint4(f32x2_to_bf16x2(g[0], g[1]), f32x2_to_bf16x2(g[2], g[3]),
                              f32x2_to_bf16x2(g[4], g[5]), f32x2_to_bf16x2(g[6], g[7]));
    }
  }
  }
}

// The p = 4 variants are held to the registers that keep kLossCtasPerSm CTAs per SM resident: the grid is sized
// for exactly that many, one wave.
template <bool FAST, bool GRAD, bool GRAD_F32>
__global__ void __launch_bounds__(kLossThreads, FAST ? kLossCtasPerSm : 1)
tweo_loss_kernel(const __grid_constant__ LossPtrs ptrs, const LossArgs args) {
  chain_release();   // launched in a chain: nothing of the kernel before this one is touched before the wait
  chain_wait();
  const int l = blockIdx.y;
  const uint16_t* __restrict__ a = ptrs.a[l];
  void* gptr = ptrs.g[l];
  const int64_t nvec = args.n >> 3;
  const uint4* av = reinterpret_cast<const uint4*>(a);
  const int64_t stride = (int64_t)gridDim.x * kLossThreads * kLossUnroll;
  double acc = 0.0;

  for (int64_t base = (int64_t)blockIdx.x * kLossThreads * kLossUnroll + threadIdx.x; base < nvec; base += stride) {
    uint4 v[kLossUnroll];
#pragma unroll
    for (int u = 0; u < kLossUnroll; ++u) {
      int64_t i = base + (int64_t)u * kLossThreads;
      v[u] = i < nvec ? __ldcs(av + i) : make_uint4(0, 0, 0, 0);
    }
    uint64_t acc2 = 0ull;   // (+0, +0): the a^4 terms of this iteration, two lanes (p = 4)
#pragma unroll
    for (int u = 0; u < kLossUnroll; ++u) {
      int64_t i = base + (int64_t)u * kLossThreads;
      if (i < nvec) {
        float vsum = 0.0f;
        uint4 gb;
        float4 gf[2];
        process_vec<FAST, GRAD, GRAD_F32>(v[u], args.k_grad, args.p, acc2, vsum, &gb, gf);
        if (!FAST) acc += (double)vsum;
        if (GRAD) {
          if (GRAD_F32) {
            float4* go = reinterpret_cast<float4*>(gptr) + 2 * i;
            __stcs(go, gf[0]);
            __stcs(go + 1, gf[1]);
          } else {
            __stcs(reinterpret_cast<uint4*>(gptr) + i, gb);
          }
        }
      }
    }
    if (FAST) {   // at most 16 terms per lane went into acc2 in binary32: relative error below 1e-6
      float lo, hi;
      unpack_f32x2(acc2, lo, hi);
      acc += (double)lo + (double)hi;
    }
  }
  // ragged tail (n % 8 elements), handled by the first threads of CTA 0 of this tensor
  if (blockIdx.x == 0) {
    int64_t i = (nvec << 3) + threadIdx.x;
    if (threadIdx.x < 8 && i < args.n) {
      float af = __uint_as_float((uint32_t)a[i] << 16);
      float t, g;
      if (FAST) {
        float s = af * af;
        t = s * s;
        g = __fmul_rn(args.k_grad, s * af);
      } else {
        double m = fabs((double)af);
        t = (float)pow(m, (double)args.p);
        g = af == 0.0f ? 0.0f : (float)((double)args.k_grad * copysign(pow(m, (double)args.p - 1.0), (double)af));
      }
      acc += (double)t;
      if (GRAD) {
        if (GRAD_F32) reinterpret_cast<float*>(gptr)[i] = g;
        else reinterpret_cast<uint16_t*>(gptr)[i] = (uint16_t)f32_to_bf16_bits(g);
      }
    }
  }

  // CTA reduction in a fixed order; one partial per CTA
  __shared__ double warp_part[kLossThreads / 32];
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < kLossThreads / 32; ++w) s += warp_part[w];
    args.partials[(size_t)l * gridDim.x + blockIdx.x] = s;
  }
}

// One CTA: warp w sums the partials of tensors w, w + 8, ... -- every lane a strided share with eight
// independent loads in flight (one round trip to L2), then a fixed shuffle tree -- and thread 0 takes the mean
// over the L tensors.  The order depends on the grid of the streaming kernel only.
__global__ void __launch_bounds__(kLossThreads) tweo_loss_finish_kernel(const LossArgs args) {
  chain_release();
  chain_wait();   // the streaming kernel has completed: its partial sums are visible
  __shared__ double block_loss[TWEO_MAX_BLOCKS];
  const int lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;
  const unsigned int parts = (unsigned int)args.parts_per_tensor;
  for (int t = wrp; t < args.L; t += kLossThreads / 32) {
    const double* part = args.partials + (size_t)t * parts;
    double s = 0.0;
    for (unsigned int b0 = lane; b0 < parts; b0 += 32 * 8) {
      double v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const unsigned int b = b0 + 32u * j;
        v[j] = b < parts ? __ldcg(part + b) : 0.0;
      }
      s += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
    }
    s = warp_sum(s);
    if (lane == 0) block_loss[t] = s * args.inv_norm;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double sum = 0.0;
    for (int t = 0; t < args.L; ++t) {
      sum += block_loss[t];
      if (args.loss_per_block) args.loss_per_block[t] = (float)block_loss[t];
    }
    *args.loss = (float)(sum / (double)args.L);
  }
}

template <bool FAST, bool GRAD, bool GRAD_F32>
void launch(dim3 grid, cudaStream_t st, const LossPtrs& ptrs, const LossArgs& args) {
  launch_chain(tweo_loss_kernel<FAST, GRAD, GRAD_F32>, grid, dim3(kLossThreads), 0, st, 0, ptrs, args);
}

// Argument checks, kernel arguments and launch shared by the two entry points; they differ only in where the
// scratch memory (partial sums from byte 256; every one that is read was written by the same call) lives.
tweo_status_t check_loss_args(const uint16_t* const* a, int32_t L, int64_t n_per_tensor, float tau, float eps, float p,
                              const float* loss, void* const* grad, int32_t grad_dtype) {
  if (!a || !loss || L < 1 || L > TWEO_MAX_BLOCKS || n_per_tensor < 0) return TWEO_ERR_INVALID_ARG;
  if (!(p > 1.0f) || !(tau + eps > 0.0f)) return TWEO_ERR_INVALID_ARG;
  if (grad && grad_dtype != TWEO_BF16 && grad_dtype != TWEO_F32) return TWEO_ERR_INVALID_ARG;
  for (int l = 0; l < L; ++l) {
    if (!a[l] && n_per_tensor > 0) return TWEO_ERR_INVALID_ARG;
    if (!aligned16(a[l])) return TWEO_ERR_ALIGNMENT;
    if (grad) {
      if (!grad[l] && n_per_tensor > 0) return TWEO_ERR_INVALID_ARG;
      if (!aligned16(grad[l])) return TWEO_ERR_ALIGNMENT;
      if (grad_dtype == TWEO_F32 && grad[l] == (const void*)a[l] && n_per_tensor > 0) return TWEO_ERR_INVALID_ARG;
    }
  }
  return TWEO_OK;
}

tweo_status_t launch_loss(const uint16_t* const* a, int32_t L, int64_t n_per_tensor, float tau, float eps, float p,
                          float grad_coeff, float* loss, float* loss_per_block, void* const* grad, int32_t grad_dtype,
                          void* scratch, int blocks_per_tensor, cudaStream_t st, const char* what) {
  LossPtrs ptrs;
  for (int l = 0; l < L; ++l) {
    ptrs.a[l] = a[l];
    ptrs.g[l] = grad ? grad[l] : nullptr;
  }
  LossArgs args;
  args.n = n_per_tensor;
  args.L = L;
  args.p = p;
  const double d = (double)tau + (double)eps;
  const double norm = (double)n_per_tensor * pow(d, (double)p);
  args.inv_norm = n_per_tensor > 0 ? 1.0 / norm : 0.0;
  args.k_grad = n_per_tensor > 0 ? (float)((double)grad_coeff * (double)p / norm) : 0.0f;
  args.loss = loss;
  args.loss_per_block = loss_per_block;
  args.partials = reinterpret_cast<double*>(reinterpret_cast<char*>(scratch) + 256);
  args.parts_per_tensor = blocks_per_tensor;

  dim3 grid((unsigned)blocks_per_tensor, (unsigned)L);
  const bool fast = (p == 4.0f);
  const bool has_grad = grad != nullptr;
  const bool f32 = grad_dtype == TWEO_F32;
  if (fast) {
    if (!has_grad) launch<true, false, false>(grid, st, ptrs, args);
    else if (f32) launch<true, true, true>(grid, st, ptrs, args);
    else launch<true, true, false>(grid, st, ptrs, args);
  } else {
    if (!has_grad) launch<false, false, false>(grid, st, ptrs, args);
    else if (f32) launch<false, true, true>(grid, st, ptrs, args);
    else launch<false, true, false>(grid, st, ptrs, args);
  }
  launch_chain(tweo_loss_finish_kernel, dim3(1), dim3(kLossThreads), 0, st, 0, args);
  tweo_detail::count_launch(2);
  return tweo_detail::check_launch(what);
}

}  // namespace

extern "C" tweo_status_t tweo_loss_fwd_bwd(const uint16_t* const* a, int32_t L, int64_t n_per_tensor, float tau,
                                           float eps, float p, float grad_coeff, float* loss,
                                           float* loss_per_block, void* const* grad, int32_t grad_dtype,
                                           void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_loss_fwd_bwd " "L=%d n=%lld tau=%g eps=%g p=%g c=%g grad=%p grad_dtype=%d ws_bytes=%zu", L,(long long)n_per_tensor,(double)tau,(double)eps,(double)p,(double)grad_coeff,(const void*)grad,grad_dtype,ws_bytes);
  tweo_status_t s = check_loss_args(a, L, n_per_tensor, tau, eps, p, loss, grad, grad_dtype);
  if (s != TWEO_OK) return s;
  const size_t need = tweo_workspace_bytes(TWEO_OP_LOSS, n_per_tensor, L, 0);
  if (!ws || ws_bytes < need) return TWEO_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(ws)) return TWEO_ERR_ALIGNMENT;
  return launch_loss(a, L, n_per_tensor, tau, eps, p, grad_coeff, loss, loss_per_block, grad, grad_dtype, ws,
                     tweo_detail::loss_blocks_per_tensor(n_per_tensor, L), (cudaStream_t)stream, "tweo_loss_kernel");
}

// ---------------------------------------------------------------------------------------
// Variant of the entry point above for callers that cannot allocate device memory.
//
// The partial sums live in a fixed array inside the library image
// instead of a caller-provided workspace.  Every GPU that loads the library holds these
// 33 KB until the process exits.  The kernel is the one above, unchanged.
namespace {

constexpr size_t kStaticPartials = 4096;                                   // partial sums that fit
constexpr size_t kStaticScratchBytes = 256 + sizeof(double) * kStaticPartials;  // 33024 bytes

static __device__ __align__(256) unsigned char g_loss_static_scratch[kStaticScratchBytes];

// In host code the array's name is only a handle for the runtime, not a device address:
// the real address is looked up once per device, with that device current.
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_static_scratch_mutex;

tweo_status_t static_scratch_for_current_device(void** out) {
  int dev = -1;
  TWEO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return TWEO_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[dev]) {
    void* ptr = nullptr;
    TWEO_CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_loss_static_scratch));
    if (!ptr) return TWEO_ERR_CUDA;
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return TWEO_OK;
}

}  // namespace

extern "C" tweo_status_t tweo_loss_fwd_bwd_static(const uint16_t* const* a, int32_t L, int64_t n_per_tensor,
                                                  float tau, float eps, float p, float grad_coeff, float* loss,
                                                  float* loss_per_block, void* const* grad, int32_t grad_dtype,
                                                  void* stream) {
  tweo_status_t s = check_loss_args(a, L, n_per_tensor, tau, eps, p, loss, grad, grad_dtype);
  if (s != TWEO_OK) return s;
  const int blocks = tweo_detail::loss_blocks_per_tensor(n_per_tensor, L);
  if ((size_t)blocks * (size_t)L > kStaticPartials) {
    // more partial sums than the built-in scratch holds: use tweo_loss_fwd_bwd with a workspace
    return TWEO_ERR_WORKSPACE_TOO_SMALL;
  }
  void* scratch = nullptr;
  s = static_scratch_for_current_device(&scratch);
  if (s != TWEO_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps whatever the previous call left.  Nothing in it has to start at zero: the streaming kernel
  // overwrites every partial sum the finishing kernel reads.
  return launch_loss(a, L, n_per_tensor, tau, eps, p, grad_coeff, loss, loss_per_block, grad, grad_dtype, scratch,
                     blocks, st, "tweo_loss_kernel (static scratch)");
}
