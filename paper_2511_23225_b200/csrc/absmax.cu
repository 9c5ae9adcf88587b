// Symmetric AbsMax b-bit quantisation (Eq. 4): s = max|X| + eps, X_q = round(X / s * Q_b),
// Q_b = 2^(b-1) - 1, with one s per tensor or per row (per output channel of a weight, per
// token of an activation), computed now or given (static).  Codes are int8 (b = 6 uses the
// same container).  Everything is binary32, each operation rounded once; Eq. 4's X / s * Q_b is
// evaluated as X * (Q_b / s), one division per scale and one multiplication per element:
//   s = fl32(amax + eps);  c = fl32(Q_b / s);  q = clamp(rne_int(fl32(x * c)), -Q_b, Q_b);  NaN -> 0.
// HBM-bound streaming kernels: 16-byte loads of 8 bf16, 16-byte stores of 16 codes.
//   per row   : one CTA per row (grid-stride over rows): maximum of the row, then the cast;
//               the second read of the row comes from L1/L2.
//   per tensor: kernel 1 writes per-CTA maxima to workspace slots, kernel 2 reduces them in
//               every CTA and casts (no atomics, no reset kernel); static s skips kernel 1.
#include <cuda_runtime.h>

#include "common.cuh"

namespace {

using namespace tweo_detail;

constexpr int kThreads = 256;
constexpr int kMaxSlots = 2048;

__device__ __forceinline__ uint32_t cta_max_bits(uint32_t m, uint32_t* part) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
  __syncthreads();
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) m = max(m, part[w]);
  return m;
}

// c = fl32(Q / s)
__device__ __forceinline__ int quant1(float x, float c, float Q) {
  const int r = __float2int_rn(__fmul_rn(x, c));  // ties to even; NaN -> 0; saturates
  const int q = (int)Q;
  return max(-q, min(q, r));
}

// 16 bf16 (two 16-byte vectors) -> 16 int8 codes
__device__ __forceinline__ uint4 quant16(const uint4 a, const uint4 b, float c, float Q) {
  const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
  uint32_t pk[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int q0 = quant1(bf16lo_to_f32(w[2 * j]), c, Q), q1 = quant1(bf16hi_to_f32(w[2 * j]), c, Q);
    const int q2 = quant1(bf16lo_to_f32(w[2 * j + 1]), c, Q), q3 = quant1(bf16hi_to_f32(w[2 * j + 1]), c, Q);
    pk[j] = (uint32_t)(q0 & 0xFF) | ((uint32_t)(q1 & 0xFF) << 8) | ((uint32_t)(q2 & 0xFF) << 16) |
           ((uint32_t)(q3 & 0xFF) << 24);
  }
  return make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// maximum of |x| over [x, x+n) by this CTA's threads (packed lanes, see absmax_bits)
__device__ __forceinline__ uint32_t span_absmax(const uint16_t* x, int64_t n, int64_t first_vec, int64_t vec_stride) {
  uint32_t m2 = 0;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
  const int64_t nvec = vec_ok ? (n >> 3) : 0;
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  for (int64_t i = first_vec; i < nvec; i += vec_stride) {
    const uint4 v = __ldg(xv + i);
    m2 = absmax_bits(m2, v.x);
    m2 = absmax_bits(m2, v.y);
    m2 = absmax_bits(m2, v.z);
    m2 = absmax_bits(m2, v.w);
  }
  for (int64_t i = (nvec << 3) + first_vec; i < n; i += vec_stride) m2 = absmax_bits(m2, (uint32_t)x[i]);
  return m2;
}

__device__ __forceinline__ void span_quantize(const uint16_t* x, int8_t* q, int64_t n, float s, float Q,
                                              int64_t first, int64_t stride) {
  const float c = __fdiv_rn(Q, s);
  const bool vec_ok = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(q)) & 15u) == 0;
  const int64_t n16 = vec_ok ? (n >> 4) : 0;
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  uint4* qv = reinterpret_cast<uint4*>(q);
  for (int64_t i = first; i < n16; i += 2 * stride) {  // two groups of 16 per iteration: four loads in flight
    const int64_t i1 = i + stride;
    const uint4 a0 = __ldcs(xv + 2 * i), b0 = __ldcs(xv + 2 * i + 1);
    uint4 a1 = a0, b1 = b0;
    if (i1 < n16) {
      a1 = __ldcs(xv + 2 * i1);
      b1 = __ldcs(xv + 2 * i1 + 1);
    }
    __stcs(qv + i, quant16(a0, b0, c, Q));
    if (i1 < n16) __stcs(qv + i1, quant16(a1, b1, c, Q));
  }
  for (int64_t i = (n16 << 4) + first; i < n; i += stride)
    q[i] = (int8_t)quant1(bf16lo_to_f32((uint32_t)x[i]), c, Q);
}

// one scale per row
template <bool GIVEN>
__global__ void __launch_bounds__(kThreads)
absmax_rows_kernel(const uint16_t* x, int64_t rows, int64_t cols, int64_t ldx, float eps, float Q, float* s_out,
                   int8_t* q, int64_t ldq) {
  __shared__ uint32_t part[kThreads / 32];
  for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const uint16_t* xr = x + r * ldx;
    float s;
    if (GIVEN) {
      s = __ldg(s_out + r);
    } else {
      const uint32_t m = cta_max_bits(absmax_fold(span_absmax(xr, cols, threadIdx.x, kThreads)), part);
      s = __fadd_rn(__uint_as_float(m << 16), eps);
      if (threadIdx.x == 0) s_out[r] = s;
    }
    span_quantize(xr, q + r * ldq, cols, s, Q, threadIdx.x, kThreads);
  }
}

// one scale for the whole (contiguous) tensor: per-CTA maxima ...
__global__ void __launch_bounds__(kThreads) absmax_slots_kernel(const uint16_t* x, int64_t n, uint32_t* slots) {
  __shared__ uint32_t part[kThreads / 32];
  const uint32_t m = cta_max_bits(
      absmax_fold(span_absmax(x, n, (int64_t)blockIdx.x * kThreads + threadIdx.x, (int64_t)gridDim.x * kThreads)), part);
  if (threadIdx.x == 0) slots[blockIdx.x] = m;
}

// ... then every CTA reduces them itself and casts its share
template <bool GIVEN>
__global__ void __launch_bounds__(kThreads)
absmax_tensor_kernel(const uint16_t* x, int64_t n, float eps, float Q, float* s_io, const uint32_t* slots, int n_slots,
                     int8_t* q) {
  __shared__ uint32_t part[kThreads / 32];
  float s;
  if (GIVEN) {
    s = __ldg(s_io);
  } else {
    uint32_t m = 0;
    for (int k = threadIdx.x; k < n_slots; k += kThreads) m = max(m, __ldcg(slots + k));
    m = cta_max_bits(m, part);
    s = __fadd_rn(__uint_as_float(m << 16), eps);
    if (blockIdx.x == 0 && threadIdx.x == 0) *s_io = s;
  }
  span_quantize(x, q, n, s, Q, (int64_t)blockIdx.x * kThreads + threadIdx.x, (int64_t)gridDim.x * kThreads);
}

int grid_cap(int64_t want, int per_sm) {
  return balanced_grid(want, (int64_t)sm_count() * per_sm);
}

}  // namespace

namespace tweo_detail {
size_t absmax_workspace_bytes() { return (size_t)kMaxSlots * sizeof(uint32_t); }
}

extern "C" tweo_status_t tweo_absmax_quantize(const uint16_t* x, int64_t rows, int64_t cols, int64_t ldx, int32_t bits,
                                              int32_t granularity, int32_t mode, float eps, float* s, int8_t* q,
                                              int64_t ldq, void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_absmax_quantize " "rows=%lld cols=%lld ldx=%lld bits=%d", (long long)rows,(long long)cols,(long long)ldx,bits);
  if (rows < 0 || cols < 0 || !s) return TWEO_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return TWEO_ERR_INVALID_ARG;
  if (granularity != TWEO_GRAN_TENSOR && granularity != TWEO_GRAN_ROW) return TWEO_ERR_INVALID_ARG;
  if (mode != TWEO_SCALE_CURRENT && mode != TWEO_SCALE_GIVEN) return TWEO_ERR_INVALID_ARG;
  if (!(eps >= 0.0f)) return TWEO_ERR_INVALID_ARG;
  if (rows * cols > 0 && (!x || !q || ldx < cols || ldq < cols)) return TWEO_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const float Q = (float)((1 << (bits - 1)) - 1);
  const bool given = mode == TWEO_SCALE_GIVEN;
  if (granularity == TWEO_GRAN_ROW) {
    if (rows == 0) return TWEO_OK;
    const int grid = grid_cap(rows, 8);
    if (given) absmax_rows_kernel<true><<<grid, kThreads, 0, st>>>(x, rows, cols, ldx, eps, Q, s, q, ldq);
    else absmax_rows_kernel<false><<<grid, kThreads, 0, st>>>(x, rows, cols, ldx, eps, Q, s, q, ldq);
    count_launch();
    return check_launch("absmax_rows_kernel");
  }
  if (rows > 1 && (ldx != cols || ldq != cols)) return TWEO_ERR_UNSUPPORTED_SHAPE;  // one scale: dense tensor
  const int64_t n = rows * cols;
  uint32_t* slots = reinterpret_cast<uint32_t*>(ws);
  int n_slots = 0;
  if (!given) {
    if (!ws || ws_bytes < absmax_workspace_bytes()) return TWEO_ERR_WORKSPACE_TOO_SMALL;
    if (!aligned16(ws)) return TWEO_ERR_ALIGNMENT;
    n_slots = grid_cap(((n >> 3) + kThreads * 4 - 1) / (kThreads * 4), 8);
    if (n_slots > kMaxSlots) n_slots = kMaxSlots;
    absmax_slots_kernel<<<n_slots, kThreads, 0, st>>>(x, n, slots);
    count_launch();
  }
  const int grid = grid_cap(((n >> 4) + kThreads * 2 - 1) / (kThreads * 2), 8);
  if (given) absmax_tensor_kernel<true><<<grid, kThreads, 0, st>>>(x, n, eps, Q, s, slots, n_slots, q);
  else absmax_tensor_kernel<false><<<grid, kThreads, 0, st>>>(x, n, eps, Q, s, slots, n_slots, q);
  count_launch();
  return check_launch("absmax_tensor_kernel");
}

// ------------------------------------------------------------------ 8-bit residual stream (Sec. 4.4)
// yq = clamp(rne_int(xq * (sx / sy) + fq * (sf / sy))): Eq. 4 dequantise, add, Eq. 4 quantise with Q_b
// cancelled.  2 bytes read and 1 written per element, 16 codes per 16-byte vector, four vectors of each
// input in flight per thread; one product, one fused multiply-add and three conversions per element.
namespace {

__device__ __forceinline__ float code_to_f32(uint32_t w, int e) { return (float)(int)(int8_t)(w >> (8 * e)); }

__device__ __forceinline__ int add1_q8(float x, float f, float a, float b, int q) {
  const int r = __float2int_rn(__fmaf_rn(f, b, __fmul_rn(x, a)));  // ties to even; NaN -> 0; saturates
  return max(-q, min(q, r));
}

__device__ __forceinline__ uint32_t add4_q8(uint32_t xw, uint32_t fw, float a, float b, int q) {
  uint32_t out = 0u;
#pragma unroll
  for (int e = 0; e < 4; ++e) out |= ((uint32_t)add1_q8(code_to_f32(xw, e), code_to_f32(fw, e), a, b, q) & 0xFFu) << (8 * e);
  return out;
}

__global__ void __launch_bounds__(256) residual_add_q8_kernel(const int8_t* xq, const int8_t* fq,  // yq may alias either
                                                              int8_t* yq, int64_t n, float Q,
                                                              const float* __restrict__ sx, const float* __restrict__ sf,
                                                              const float* __restrict__ sy) {
  const float a = __fdiv_rn(__ldg(sx), __ldg(sy)), b = __fdiv_rn(__ldg(sf), __ldg(sy));
  const int q = (int)Q;
  const int64_t nvec = n >> 4;
  const uint4* xv = reinterpret_cast<const uint4*>(xq);
  const uint4* fv = reinterpret_cast<const uint4*>(fq);
  uint4* yv = reinterpret_cast<uint4*>(yq);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < nvec; i += 4 * stride) {
    uint4 va[4], vb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      va[u] = __ldcs(xv + i + u * stride);
      vb[u] = __ldcs(fv + i + u * stride);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      __stcs(yv + i + u * stride, make_uint4(add4_q8(va[u].x, vb[u].x, a, b, q), add4_q8(va[u].y, vb[u].y, a, b, q),
                                             add4_q8(va[u].z, vb[u].z, a, b, q), add4_q8(va[u].w, vb[u].w, a, b, q)));
  }
  for (; i < nvec; i += stride) {
    const uint4 va = __ldcs(xv + i), vb = __ldcs(fv + i);
    __stcs(yv + i, make_uint4(add4_q8(va.x, vb.x, a, b, q), add4_q8(va.y, vb.y, a, b, q),
                              add4_q8(va.z, vb.z, a, b, q), add4_q8(va.w, vb.w, a, b, q)));
  }
  // ragged tail (n % 16 codes) by the first threads of the grid
  const int64_t t = (nvec << 4) + (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) {
    yq[t] = (int8_t)add1_q8((float)xq[t], (float)fq[t], a, b, q);
  }
}

}  // namespace

extern "C" tweo_status_t tweo_residual_add_q8(const int8_t* xq, const float* sx, const int8_t* fq, const float* sf,
                                              int64_t n, int32_t bits, const float* sy, int8_t* yq, void* stream) {
  TWEO_LOG_CALL("tweo_residual_add_q8 " "n=%lld bits=%d", (long long)n,bits);
  if (n < 0 || bits < 2 || bits > 8 || !sx || !sf || !sy) return TWEO_ERR_INVALID_ARG;
  if (n == 0) return TWEO_OK;
  if (!xq || !fq || !yq) return TWEO_ERR_INVALID_ARG;
  if (!tweo_detail::aligned16(xq) || !tweo_detail::aligned16(fq) || !tweo_detail::aligned16(yq)) return TWEO_ERR_ALIGNMENT;
  const float Q = (float)((1 << (bits - 1)) - 1);
  const int64_t nvec = n >> 4;
  const int64_t want = (nvec + 4 * 256 - 1) / (4 * 256);
  const int grid = tweo_detail::balanced_grid(want, (int64_t)tweo_detail::sm_count() * 8);
  residual_add_q8_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(xq, fq, yq, n, Q, sx, sf, sy);
  tweo_detail::count_launch();
  return tweo_detail::check_launch("residual_add_q8_kernel");
}

// ------------------------------------------------------------------ per-token 8-bit residual stream (Sec. 4.4)
// One warp per row: the row's codes of x and f(x) stay in registers (VPL 16-byte vectors of each per lane,
// lane-interleaved), so the dequantised sum is formed once, its maximum found by shuffles, and the codes of the
// sum written in the same pass: 2 bytes read and 1 written per element plus three scales per row.
namespace {

struct RowAddArgs {
  const int8_t* xq;
  const int8_t* fq;
  int8_t* yq;
  const float* sx;
  const float* sf;
  float* sy;
  int64_t rows;
  int32_t cols;
  float Q, eps;
};

template <int VPL>
__global__ void __launch_bounds__(256) residual_add_q8_rows_kernel(const RowAddArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t warp_global = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * 8;
  const int nvec = a.cols >> 4;
  const int q = (int)a.Q;
  for (int64_t row = warp_global; row < a.rows; row += warp_stride) {
    const uint4* xv = reinterpret_cast<const uint4*>(a.xq + row * a.cols);
    const uint4* fv = reinterpret_cast<const uint4*>(a.fq + row * a.cols);
    uint4 vx[VPL], vf[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      const int idx = lane + 32 * i;
      vx[i] = idx < nvec ? __ldcs(xv + idx) : make_uint4(0u, 0u, 0u, 0u);
      vf[i] = idx < nvec ? __ldcs(fv + idx) : make_uint4(0u, 0u, 0u, 0u);
    }
    const float cx = __fdiv_rn(__ldg(a.sx + row), a.Q), cf = __fdiv_rn(__ldg(a.sf + row), a.Q);
    float amax = 0.0f;  // padding lanes hold zero codes: their sum is 0
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      const uint32_t wx[4] = {vx[i].x, vx[i].y, vx[i].z, vx[i].w};
      const uint32_t wf[4] = {vf[i].x, vf[i].y, vf[i].z, vf[i].w};
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          amax = fmaxf(amax, fabsf(__fmaf_rn(code_to_f32(wf[k], e), cf, __fmul_rn(code_to_f32(wx[k], e), cx))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
    const float s = __fadd_rn(amax, a.eps);
    const float c = __fdiv_rn(a.Q, s);
    if (lane == 0) a.sy[row] = s;
    uint4* yv = reinterpret_cast<uint4*>(a.yq + row * a.cols);
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      const int idx = lane + 32 * i;
      if (idx < nvec) {
        const uint32_t wx[4] = {vx[i].x, vx[i].y, vx[i].z, vx[i].w};
        const uint32_t wf[4] = {vf[i].x, vf[i].y, vf[i].z, vf[i].w};
        uint32_t o4[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          uint32_t w = 0u;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float y = __fmaf_rn(code_to_f32(wf[k], e), cf, __fmul_rn(code_to_f32(wx[k], e), cx));
            w |= ((uint32_t)quant1(y, c, a.Q) & 0xFFu) << (8 * e);
          }
          o4[k] = w;
        }
        __stcs(yv + idx, make_uint4(o4[0], o4[1], o4[2], o4[3]));
      }
    }
    (void)q;
  }
}

template <int VPL>
cudaError_t launch_row_add(const RowAddArgs& a, cudaStream_t st) {
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, residual_add_q8_rows_kernel<VPL>, 256, 0);
  if (e != cudaSuccess) return e;
  const int64_t want = (a.rows + 7) / 8;
  const int64_t cap = (int64_t)tweo_detail::sm_count() * (per_sm > 0 ? per_sm : 1);
  residual_add_q8_rows_kernel<VPL><<<tweo_detail::balanced_grid(want, cap), 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

extern "C" tweo_status_t tweo_residual_add_q8_rows(const int8_t* xq, const float* sx, const int8_t* fq, const float* sf,
                                                   int64_t rows, int64_t cols, int32_t bits, float eps, int8_t* yq,
                                                   float* sy, void* stream) {
  TWEO_LOG_CALL("tweo_residual_add_q8_rows " "rows=%lld cols=%lld bits=%d eps=%g", (long long)rows,(long long)cols,bits,(double)eps);
  if (rows < 0 || cols < 1 || bits < 2 || bits > 8 || !(eps >= 0.0f)) return TWEO_ERR_INVALID_ARG;
  if ((cols & 15) || cols > 8192) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (rows == 0) return TWEO_OK;
  if (!xq || !fq || !yq || !sx || !sf || !sy) return TWEO_ERR_INVALID_ARG;
  if (!tweo_detail::aligned16(xq) || !tweo_detail::aligned16(fq) || !tweo_detail::aligned16(yq)) return TWEO_ERR_ALIGNMENT;
  RowAddArgs a;
  a.xq = xq;
  a.fq = fq;
  a.yq = yq;
  a.sx = sx;
  a.sf = sf;
  a.sy = sy;
  a.rows = rows;
  a.cols = (int32_t)cols;
  a.Q = (float)((1 << (bits - 1)) - 1);
  a.eps = eps;
  cudaStream_t st = (cudaStream_t)stream;
  const int vpl = (int)((cols / 16 + 31) / 32);
  cudaError_t e;
  if (vpl <= 1) e = launch_row_add<1>(a, st);
  else if (vpl <= 2) e = launch_row_add<2>(a, st);
  else if (vpl <= 4) e = launch_row_add<4>(a, st);
  else if (vpl <= 8) e = launch_row_add<8>(a, st);
  else e = launch_row_add<16>(a, st);
  if (e != cudaSuccess) return tweo_detail::cuda_fail(e, "residual_add_q8_rows_kernel");
  tweo_detail::count_launch();
  return TWEO_OK;
}
