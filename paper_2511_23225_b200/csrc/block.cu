// Block output in one pass, and the delayed-scaling state update.
//
// (1) The TWEO penalty acts on the output of every transformer block, A = x + f(x) (Sec. 3.3),
// and with delayed per-tensor scaling (Sec. 4.3) the scale of A for the next block's FP8
// linears is known before A exists.  So everything that touches A once can ride on the
// residual addition itself: read x and f, form a = bf16(fl32(x + f)), and in the same pass
// emit a, the penalty's partial sums, its gradient, amax(a) and the FP8 codes of a.  That is
// 4 B read + up to 5 B written per element instead of the 13 B of add, penalty and cast as
// three passes.  HBM-bound streaming kernel: 8 x 16-byte loads in flight per thread (two groups of 16 elements),
// fp32 per group / fp64 per thread accumulation, per-CTA partial sum and partial maximum to
// the workspace; a one-CTA kernel launched in the same chain reduces them in a fixed order (the
// streaming CTAs end without fence, ticket or wait: see loss.cu).
//
// (2) One tiny kernel keeps the amax history of every tensor (length H, 16 in the paper) and
// derives next step's scales from the maximum over the window.
#include <cuda_runtime.h>

#include "common.cuh"

namespace {

using namespace tweo_detail;

constexpr int kThreads = 256;

struct BlockArgs {
  const uint16_t* x;
  const uint16_t* f;
  uint16_t* a;
  uint16_t* g;        // or nullptr
  uint8_t* q;         // or nullptr
  const float* q_scale;
  int64_t n;
  float p;
  float k_grad;       // fl32(grad_coeff * p / (n * (tau+eps)^p)), rounded once on the host
  double inv_norm;    // 1 / (n * (tau+eps)^p)
  float* loss;
  float* amax;
  double* part_sum;   // [grid]
  uint32_t* part_max; // [grid]
  int parts;          // grid of the streaming kernel
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
  return v;
}

// One pair of elements: returns the packed bf16 sum, adds |a|^p of both to t, and (GRAD) packs the gradients.
template <bool FAST, bool GRAD>
__device__ __forceinline__ uint32_t add_pair(uint32_t xw, uint32_t fw, float k, float p, float& t, uint32_t& gw) {
  const float s0 = __fadd_rn(bf16lo_to_f32(xw), bf16lo_to_f32(fw));
  const float s1 = __fadd_rn(bf16hi_to_f32(xw), bf16hi_to_f32(fw));
  const uint32_t aw = f32x2_to_bf16x2(s0, s1);
  const float a0 = bf16lo_to_f32(aw), a1 = bf16hi_to_f32(aw);
  float g0, g1;
  if (FAST) {
    const float q0 = a0 * a0, q1 = a1 * a1;
    t += q0 * q0 + q1 * q1;
    if (GRAD) {
      g0 = __fmul_rn(k, q0 * a0);
      g1 = __fmul_rn(k, q1 * a1);
    }
  } else {
    const double m0 = fabs((double)a0), m1 = fabs((double)a1);
    t += (float)pow(m0, (double)p) + (float)pow(m1, (double)p);
    if (GRAD) {
      g0 = a0 == 0.0f ? 0.0f : (float)((double)k * copysign(pow(m0, (double)p - 1.0), (double)a0));
      g1 = a1 == 0.0f ? 0.0f : (float)((double)k * copysign(pow(m1, (double)p - 1.0), (double)a1));
    }
  }
  if (GRAD) gw = f32x2_to_bf16x2(g0, g1);
  return aw;
}

// QFMT: -1 no FP8 copy, else TWEO_E4M3 / TWEO_E5M2
template <bool FAST, bool GRAD, int QFMT>
__global__ void __launch_bounds__(kThreads) block_output_kernel(const BlockArgs args) {
  chain_release();   // launched in a chain: nothing of the kernel before this one is touched before the wait
  chain_wait();
  const int64_t n16 = args.n >> 4;
  const uint4* xv = reinterpret_cast<const uint4*>(args.x);
  const uint4* fv = reinterpret_cast<const uint4*>(args.f);
  uint4* av = reinterpret_cast<uint4*>(args.a);
  uint4* gv = reinterpret_cast<uint4*>(args.g);
  uint4* qv = reinterpret_cast<uint4*>(args.q);
  const float qs = QFMT >= 0 ? __ldg(args.q_scale) : 0.0f;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  double acc = 0.0;
  uint32_t m2 = 0;
  // two groups of 16 elements per thread and iteration: eight 16-byte loads in flight
  for (int64_t base = (int64_t)blockIdx.x * kThreads + threadIdx.x; base < n16; base += 2 * stride) {
    uint4 xr[2][2], fr[2][2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int64_t i = base + u * stride;
      if (i < n16) {
        xr[u][0] = __ldcs(xv + 2 * i);
        xr[u][1] = __ldcs(xv + 2 * i + 1);
        fr[u][0] = __ldcs(fv + 2 * i);
        fr[u][1] = __ldcs(fv + 2 * i + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int64_t i = base + u * stride;
      if (i >= n16) continue;
      const uint32_t xw[8] = {xr[u][0].x, xr[u][0].y, xr[u][0].z, xr[u][0].w, xr[u][1].x, xr[u][1].y, xr[u][1].z, xr[u][1].w};
      const uint32_t fw[8] = {fr[u][0].x, fr[u][0].y, fr[u][0].z, fr[u][0].w, fr[u][1].x, fr[u][1].y, fr[u][1].z, fr[u][1].w};
      uint32_t aw[8], gw[8], c[8];
      float t = 0.0f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        aw[j] = add_pair<FAST, GRAD>(xw[j], fw[j], args.k_grad, args.p, t, gw[j]);
        m2 = absmax_bits(m2, aw[j]);
      }
      acc += (double)t;
      __stcs(av + 2 * i, make_uint4(aw[0], aw[1], aw[2], aw[3]));
      __stcs(av + 2 * i + 1, make_uint4(aw[4], aw[5], aw[6], aw[7]));
      if (GRAD) {
        __stcs(gv + 2 * i, make_uint4(gw[0], gw[1], gw[2], gw[3]));
        __stcs(gv + 2 * i + 1, make_uint4(gw[4], gw[5], gw[6], gw[7]));
      }
      if (QFMT >= 0) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float lo = __fmul_rn(bf16lo_to_f32(aw[j]), qs), hi = __fmul_rn(bf16hi_to_f32(aw[j]), qs);
          c[j] = cvt_fp8x2<QFMT < 0 ? 0 : QFMT>(lo, hi);
        }
        __stcs(qv + i, make_uint4(c[0] | (c[1] << 16), c[2] | (c[3] << 16), c[4] | (c[5] << 16), c[6] | (c[7] << 16)));
      }
    }
  }
  // ragged tail (n % 16 elements), first threads of CTA 0
  if (blockIdx.x == 0 && threadIdx.x < 16) {
    const int64_t i = (n16 << 4) + threadIdx.x;
    if (i < args.n) {
      float t = 0.0f;
      uint32_t gw = 0;
      const uint32_t aw = add_pair<FAST, GRAD>((uint32_t)args.x[i], (uint32_t)args.f[i], args.k_grad, args.p, t, gw);
      // the upper half of the pair is 0 + 0 = 0 and contributes nothing
      acc += (double)t;
      m2 = absmax_bits(m2, aw & 0xFFFFu);
      args.a[i] = (uint16_t)(aw & 0xFFFFu);
      if (GRAD) args.g[i] = (uint16_t)(gw & 0xFFFFu);
      if (QFMT >= 0) {
        const float v = __fmul_rn(bf16lo_to_f32(aw), qs);
        args.q[i] = (uint8_t)(cvt_fp8x2<QFMT < 0 ? 0 : QFMT>(v, 0.0f) & 0xFFu);
      }
    }
  }

  // CTA reduction in a fixed order; one partial sum and one partial maximum per CTA
  __shared__ double warp_part[kThreads / 32];
  __shared__ uint32_t warp_maxv[kThreads / 32];
  acc = warp_sum(acc);
  uint32_t m = absmax_fold(m2);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0) {
    warp_part[threadIdx.x >> 5] = acc;
    warp_maxv[threadIdx.x >> 5] = m;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    uint32_t mm = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      s += warp_part[w];
      mm = max(mm, warp_maxv[w]);
    }
    args.part_sum[blockIdx.x] = s;
    args.part_max[blockIdx.x] = mm;
  }
}

// One CTA adds the partial sums (thread-strided with independent loads, then a fixed tree) and takes the maximum.
__global__ void __launch_bounds__(kThreads) block_output_finish_kernel(const BlockArgs args) {
  chain_release();
  chain_wait();   // the streaming kernel has completed: its partial results are visible
  __shared__ double warp_part[kThreads / 32];
  __shared__ uint32_t warp_maxv[kThreads / 32];
  const unsigned int parts = (unsigned int)args.parts;
  double s = 0.0;
  uint32_t mm = 0;
  for (unsigned int b0 = threadIdx.x; b0 < parts; b0 += kThreads * 4) {
    double v[4];
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const unsigned int b = b0 + (unsigned int)(kThreads * j);
      v[j] = b < parts ? __ldcg(&args.part_sum[b]) : 0.0;
      w[j] = b < parts ? __ldcg(&args.part_max[b]) : 0u;
    }
    s += (v[0] + v[1]) + (v[2] + v[3]);
    mm = max(max(mm, max(w[0], w[1])), max(w[2], w[3]));
  }
  s = warp_sum(s);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mm = max(mm, __shfl_xor_sync(0xFFFFFFFFu, mm, o));
  if ((threadIdx.x & 31) == 0) {
    warp_part[threadIdx.x >> 5] = s;
    warp_maxv[threadIdx.x >> 5] = mm;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    uint32_t mx = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      tot += warp_part[w];
      mx = max(mx, warp_maxv[w]);
    }
    *args.loss = (float)(tot * args.inv_norm);
    *args.amax = __uint_as_float(mx << 16);
  }
}

template <bool FAST, bool GRAD>
void launch_q(int qfmt, int grid, cudaStream_t st, const BlockArgs& a) {
  if (qfmt < 0) launch_chain(block_output_kernel<FAST, GRAD, -1>, dim3(grid), dim3(kThreads), 0, st, 0, a);
  else if (qfmt == TWEO_E4M3) launch_chain(block_output_kernel<FAST, GRAD, TWEO_E4M3>, dim3(grid), dim3(kThreads), 0, st, 0, a);
  else launch_chain(block_output_kernel<FAST, GRAD, TWEO_E5M2>, dim3(grid), dim3(kThreads), 0, st, 0, a);
}

int block_grid(int64_t n) {
  return balanced_grid(((n >> 4) + 2 * kThreads - 1) / (2 * kThreads), (int64_t)sm_count() * 8);
}

__global__ void delayed_scaling_kernel(float* history, int H, const float* amax_new, float* scale, float* scale_inv,
                                       int T, int fmt) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  float* h = history + (size_t)t * H;
  float m = 0.0f;
  for (int j = H - 1; j > 0; --j) {
    const float v = h[j - 1];
    h[j] = v;
    if (v > m) m = v;  // false for NaN
  }
  const float a = amax_new[t];
  h[0] = a;
  if (a > m) m = a;
  float s = scale[t];
  if (m > 0.0f && m < __int_as_float(0x7F800000)) {
    s = scale_from_amax(m, fmt);
    scale[t] = s;
  }
  scale_inv[t] = __fdiv_rn(1.0f, s);
}

}  // namespace

namespace tweo_detail {
size_t block_output_workspace_bytes() { return 256 + (size_t)sm_count() * 8 * (sizeof(double) + sizeof(uint32_t)); }
}

extern "C" tweo_status_t tweo_block_output_fused(const uint16_t* x, const uint16_t* f, int64_t n, float tau, float eps,
                                                 float p, float grad_coeff, uint16_t* a, uint16_t* grad, float* loss,
                                                 float* amax, uint8_t* aq, int32_t q_fmt, const float* q_scale,
                                                 void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_block_output_fused " "n=%lld tau=%g eps=%g p=%g c=%g grad=%p aq=%p q_fmt=%d ws_bytes=%zu", (long long)n,(double)tau,(double)eps,(double)p,(double)grad_coeff,(void*)grad,(void*)aq,q_fmt,ws_bytes);
  if (n < 0 || !loss || !amax) return TWEO_ERR_INVALID_ARG;
  if (n > 0 && (!x || !f || !a)) return TWEO_ERR_INVALID_ARG;
  if (!(p > 1.0f) || !(tau + eps > 0.0f)) return TWEO_ERR_INVALID_ARG;
  if (aq && (!q_scale || (q_fmt != TWEO_E4M3 && q_fmt != TWEO_E5M2))) return TWEO_ERR_INVALID_ARG;
  if (grad && n > 0 && (grad == a || grad == x || grad == f)) return TWEO_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(f) || !aligned16(a) || !aligned16(grad) || !aligned16(aq)) return TWEO_ERR_ALIGNMENT;
  if (!ws || ws_bytes < tweo_detail::block_output_workspace_bytes()) return TWEO_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(ws)) return TWEO_ERR_ALIGNMENT;
  const int grid = block_grid(n);
  BlockArgs args;
  args.x = x;
  args.f = f;
  args.a = a;
  args.g = grad;
  args.q = aq;
  args.q_scale = q_scale;
  args.n = n;
  args.p = p;
  const double d = (double)tau + (double)eps;
  const double norm = (double)n * pow(d, (double)p);
  args.inv_norm = n > 0 ? 1.0 / norm : 0.0;
  args.k_grad = n > 0 ? (float)((double)grad_coeff * (double)p / norm) : 0.0f;
  args.loss = loss;
  args.amax = amax;
  args.parts = grid;
  args.part_sum = reinterpret_cast<double*>(reinterpret_cast<char*>(ws) + 256);
  args.part_max = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(ws) + 256 + (size_t)sm_count() * 8 * sizeof(double));
  cudaStream_t st = (cudaStream_t)stream;
  const int qf = aq ? q_fmt : -1;
  const bool fast = p == 4.0f;
  if (fast) {
    if (grad) launch_q<true, true>(qf, grid, st, args);
    else launch_q<true, false>(qf, grid, st, args);
  } else {
    if (grad) launch_q<false, true>(qf, grid, st, args);
    else launch_q<false, false>(qf, grid, st, args);
  }
  launch_chain(block_output_finish_kernel, dim3(1), dim3(kThreads), 0, st, 0, args);
  count_launch(2);
  return check_launch("block_output_kernel");
}

extern "C" tweo_status_t tweo_delayed_scaling_update(float* amax_history, int32_t history_len, const float* amax_new,
                                                     float* scale, float* scale_inv, int32_t n_tensors, int32_t fmt,
                                                     void* stream) {
  TWEO_LOG_CALL("tweo_delayed_scaling_update " "history_len=%d n_tensors=%d fmt=%d", history_len,n_tensors,fmt);
  if (n_tensors < 0 || history_len < 1) return TWEO_ERR_INVALID_ARG;
  if (fmt != TWEO_E4M3 && fmt != TWEO_E5M2) return TWEO_ERR_INVALID_ARG;
  if (n_tensors == 0) return TWEO_OK;
  if (!amax_history || !amax_new || !scale || !scale_inv) return TWEO_ERR_INVALID_ARG;
  delayed_scaling_kernel<<<(n_tensors + 127) / 128, 128, 0, (cudaStream_t)stream>>>(amax_history, history_len, amax_new,
                                                                                   scale, scale_inv, n_tensors, fmt);
  count_launch();
  return check_launch("delayed_scaling_kernel");
}
