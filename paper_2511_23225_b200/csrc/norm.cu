// LayerNorm / RMSNorm over the last dimension with the FP8 cast of the output in the same pass.
// HBM-bound: every element is read once (2 B) and written once as bf16 (2 B) and / or FP8 (1 B).
//
// One warp per row, rows dealt round-robin to the warps of a persistent grid.  A lane holds its
// share of the row in registers (VPL 16-byte vectors, lane-interleaved so every load and store of
// the warp is contiguous), so mean, centred variance and output take one read of x.  gamma and
// beta are staged once per CTA in shared memory.  The maximum of |y| travels in registers and
// ends in one atomicMax per warp (the caller's amax is zeroed on the stream first).
#include <cuda_runtime.h>

#include "common.cuh"

namespace {

using namespace tweo_detail;

struct NormArgs {
  const uint16_t* x;
  uint16_t* y;
  uint8_t* q;
  const float* gamma;
  const float* beta;
  const float* q_scale;
  float* amax;
  float* mean;
  float* rstd;
  int64_t ldx, ldy, ldq, rows;
  int32_t d, rms, q_fmt;
  float eps;
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

constexpr int kNormThreads = 256;

// QFMT: -1 no FP8 output, else the tweo_fp8_t of the codes
template <int VPL, int QFMT>
__global__ void __launch_bounds__(kNormThreads) norm_rows_kernel(const NormArgs a) {
  extern __shared__ __align__(16) float gb[];  // gamma [d], beta [d]
  float* s_gamma = gb;
  float* s_beta = gb + a.d;
  for (int j = threadIdx.x; j < a.d; j += kNormThreads) {
    s_gamma[j] = __ldg(a.gamma + j);
    s_beta[j] = a.beta ? __ldg(a.beta + j) : 0.0f;
  }
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const int warps_per_cta = kNormThreads / 32;
  const int64_t warp_global = (int64_t)blockIdx.x * warps_per_cta + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * warps_per_cta;
  const int nvec = a.d >> 3;
  const float inv_d = 1.0f / (float)a.d;
  const float qs = QFMT >= 0 ? __ldg(a.q_scale) : 0.0f;
  float run_amax = 0.0f;

  // the next row's loads are issued before this row's reductions, so a warp always has a row in flight
  constexpr bool PREFETCH = VPL <= 8;
  uint4 nxt[PREFETCH ? VPL : 1];
  if (PREFETCH && warp_global < a.rows) {
    const uint4* xr = reinterpret_cast<const uint4*>(a.x + warp_global * a.ldx);
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      const int idx = lane + 32 * i;
      nxt[i] = idx < nvec ? __ldcs(xr + idx) : make_uint4(0u, 0u, 0u, 0u);
    }
  }
  for (int64_t row = warp_global; row < a.rows; row += warp_stride) {
    uint4 v[VPL];
    if (PREFETCH) {
#pragma unroll
      for (int i = 0; i < VPL; ++i) v[i] = nxt[i];
      const int64_t nrow = row + warp_stride;
      if (nrow < a.rows) {
        const uint4* xn = reinterpret_cast<const uint4*>(a.x + nrow * a.ldx);
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
          const int idx = lane + 32 * i;
          nxt[i] = idx < nvec ? __ldcs(xn + idx) : make_uint4(0u, 0u, 0u, 0u);
        }
      }
    } else {
      const uint4* xr = reinterpret_cast<const uint4*>(a.x + row * a.ldx);
#pragma unroll
      for (int i = 0; i < VPL; ++i) {
        const int idx = lane + 32 * i;
        v[i] = idx < nvec ? __ldcs(xr + idx) : make_uint4(0u, 0u, 0u, 0u);
      }
    }
    float mu = 0.0f;
    if (!a.rms) {
      float s = 0.0f;
#pragma unroll
      for (int i = 0; i < VPL; ++i) {
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) s += bf16lo_to_f32(w[k]) + bf16hi_to_f32(w[k]);
      }
      mu = warp_sum(s) * inv_d;
    }
    float ss = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      if (lane + 32 * i < nvec) {  // padding lanes hold zeros, which are not at distance 0 from mu
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float c0 = bf16lo_to_f32(w[k]) - mu, c1 = bf16hi_to_f32(w[k]) - mu;
          ss = fmaf(c0, c0, ss);
          ss = fmaf(c1, c1, ss);
        }
      }
    }
    const float var = warp_sum(ss) * inv_d;
    const float rs = 1.0f / sqrtf(var + a.eps);
    if (lane == 0) {
      if (a.mean) a.mean[row] = mu;
      if (a.rstd) a.rstd[row] = rs;
    }
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      const int idx = lane + 32 * i;
      if (idx < nvec) {
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        const float4 g0 = *reinterpret_cast<const float4*>(s_gamma + 8 * idx);
        const float4 g1 = *reinterpret_cast<const float4*>(s_gamma + 8 * idx + 4);
        const float4 b0 = *reinterpret_cast<const float4*>(s_beta + 8 * idx);
        const float4 b1 = *reinterpret_cast<const float4*>(s_beta + 8 * idx + 4);
        const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float y0 = fmaf((bf16lo_to_f32(w[k]) - mu) * rs, g[2 * k], b[2 * k]);
          const float y1 = fmaf((bf16hi_to_f32(w[k]) - mu) * rs, g[2 * k + 1], b[2 * k + 1]);
          o[k] = f32x2_to_bf16x2(y0, y1);
        }
        if (a.y) __stcs(reinterpret_cast<uint4*>(a.y + row * a.ldy) + idx, make_uint4(o[0], o[1], o[2], o[3]));
        if (QFMT >= 0 || a.amax) {
          float f[8];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            f[2 * k] = bf16lo_to_f32(o[k]);
            f[2 * k + 1] = bf16hi_to_f32(o[k]);
          }
          if (a.amax) {
#pragma unroll
            for (int k = 0; k < 8; ++k) run_amax = fmaxf(run_amax, fabsf(f[k]));
          }
          if (QFMT >= 0) {
            uint32_t c[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)  // NaN -> 0x7F inside cvt_fp8x2
              c[k] = cvt_fp8x2<QFMT >= 0 ? QFMT : 0>(__fmul_rn(f[2 * k], qs), __fmul_rn(f[2 * k + 1], qs));
            __stcs(reinterpret_cast<uint2*>(a.q + row * a.ldq) + idx, make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16)));
          }
        }
      }
    }
  }
  if (a.amax) {
    run_amax = warp_max(run_amax);
    if (lane == 0 && run_amax > 0.0f) atomicMax(reinterpret_cast<unsigned int*>(a.amax), __float_as_uint(run_amax));
  }
}

template <int VPL, int QFMT>
cudaError_t launch_norm_q(const NormArgs& a, int64_t want_ctas, size_t smem, cudaStream_t st) {
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {  // gamma and beta of the widest row take 64 KB
    cudaError_t e = cudaFuncSetAttribute(norm_rows_kernel<VPL, QFMT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536);
    if (e != cudaSuccess) return e;
    device_once_done(attr_done, attr_dev);
  }
  // persistent grid: as many CTAs as are resident at once
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, norm_rows_kernel<VPL, QFMT>, kNormThreads, smem);
  if (e != cudaSuccess) return e;
  const int64_t cap = (int64_t)tweo_detail::sm_count() * (per_sm > 0 ? per_sm : 1);
  const int grid = tweo_detail::balanced_grid(want_ctas, cap);
  norm_rows_kernel<VPL, QFMT><<<grid, kNormThreads, smem, st>>>(a);
  return cudaGetLastError();
}

template <int VPL>
cudaError_t launch_norm(const NormArgs& a, int64_t want_ctas, size_t smem, cudaStream_t st) {
  if (!a.q) return launch_norm_q<VPL, -1>(a, want_ctas, smem, st);
  if (a.q_fmt == TWEO_E4M3) return launch_norm_q<VPL, TWEO_E4M3>(a, want_ctas, smem, st);
  return launch_norm_q<VPL, TWEO_E5M2>(a, want_ctas, smem, st);
}

}  // namespace

extern "C" tweo_status_t tweo_layernorm_fp8(const uint16_t* x, int64_t ldx, int64_t rows, int64_t d, int32_t kind,
                                            const float* gamma, const float* beta, float eps, uint16_t* y,
                                            int64_t ldy, uint8_t* yq, int64_t ldq, int32_t q_fmt,
                                            const float* q_scale, float* amax, float* mean, float* rstd,
                                            void* stream) {
  TWEO_LOG_CALL("tweo_layernorm_fp8 " "rows=%lld d=%lld ldx=%lld kind=%d", (long long)rows,(long long)d,(long long)ldx,kind);
  if (rows < 0 || d < 1 || !gamma || (kind != TWEO_NORM_LAYER && kind != TWEO_NORM_RMS)) return TWEO_ERR_INVALID_ARG;
  if ((d & 7) || d > 8192) return TWEO_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t st = (cudaStream_t)stream;
  if (rows == 0) {  // nothing to normalise; the maximum over no element is 0
    if (amax) TWEO_CUDA_TRY(cudaMemsetAsync(amax, 0, sizeof(float), st));
    return TWEO_OK;
  }
  if (!y && !yq) return TWEO_ERR_INVALID_ARG;
  if (yq && (!q_scale || (q_fmt != TWEO_E4M3 && q_fmt != TWEO_E5M2))) return TWEO_ERR_INVALID_ARG;
  if (!(eps >= 0.0f)) return TWEO_ERR_INVALID_ARG;
  if (!x) return TWEO_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y) || !aligned16(yq) || (ldx & 7) || (y && (ldy & 7)) || (yq && (ldq & 7)))
    return TWEO_ERR_ALIGNMENT;
  if (ldx < d || (y && ldy < d) || (yq && ldq < d)) return TWEO_ERR_INVALID_ARG;
  if (amax) TWEO_CUDA_TRY(cudaMemsetAsync(amax, 0, sizeof(float), st));
  NormArgs a;
  a.x = x;
  a.y = y;
  a.q = yq;
  a.gamma = gamma;
  a.beta = beta;
  a.q_scale = q_scale;
  a.amax = amax;
  a.mean = mean;
  a.rstd = rstd;
  a.ldx = ldx;
  a.ldy = ldy;
  a.ldq = ldq;
  a.rows = rows;
  a.d = (int32_t)d;
  a.rms = kind == TWEO_NORM_RMS;
  a.q_fmt = q_fmt;
  a.eps = eps;
  const int warps_per_cta = kNormThreads / 32;
  const int64_t want = (rows + warps_per_cta - 1) / warps_per_cta;
  const int64_t grid = want;
  const size_t smem = (size_t)d * 2 * sizeof(float);
  const int vpl = (int)((d / 8 + 31) / 32);
  cudaError_t e;
  if (vpl <= 1) e = launch_norm<1>(a, grid, smem, st);
  else if (vpl <= 2) e = launch_norm<2>(a, grid, smem, st);
  else if (vpl <= 3) e = launch_norm<3>(a, grid, smem, st);
  else if (vpl <= 4) e = launch_norm<4>(a, grid, smem, st);
  else if (vpl <= 6) e = launch_norm<6>(a, grid, smem, st);
  else if (vpl <= 8) e = launch_norm<8>(a, grid, smem, st);
  else if (vpl <= 12) e = launch_norm<12>(a, grid, smem, st);
  else if (vpl <= 16) e = launch_norm<16>(a, grid, smem, st);
  else if (vpl <= 24) e = launch_norm<24>(a, grid, smem, st);
  else e = launch_norm<32>(a, grid, smem, st);
  if (e != cudaSuccess) return tweo_detail::cuda_fail(e, "norm_rows_kernel");
  tweo_detail::count_launch();
  return TWEO_OK;
}
