// FP4 (E2M1) with one scale per tensor: the step the paper's conclusion looks ahead to, with the
// per-tensor scaling of Sec. 4.3 carried over (scale = 6 / amax, saturating round-to-nearest-even).
//
// A tensor has two forms here:
//   packed   two 4-bit codes per byte (element 2i in the low nibble), what is stored and moved;
//   carrier  one byte per element holding the E4M3 code of the SAME value.  Every E2M1 value
//            (0, 0.5, 1, 1.5, 2, 3, 4, 6 and their negatives) is an E4M3 value, so the FP8 GEMM kernels
//            (tcgen05 kind::f8f6f4 on E4M3 operands) compute the FP4 product exactly: the tensor
//            core multiplies 4-bit and 8-bit floating-point operands without block scales at the
//            same rate, so nothing is lost in throughput by feeding it carriers.
// The casts use the sm_100a converters (cvt ... e2m1x2) and are HBM-bound streaming kernels of the
// same shape as the FP8 casts: 2 bytes read, 0.5 (packed) and / or 1 (carrier) written per element.
#include "common.cuh"

namespace tweo_detail {
tweo_status_t gemm_fwd_codes(const uint8_t* xq, int64_t ldx, int fmt_x, const uint8_t* wq, int64_t ldw, int fmt_w,
                             const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                             int64_t N, int64_t K, const tweo_epilogue_t* epi, void* ws, size_t ws_bytes,
                             cudaStream_t st, bool sx_is_scale);
// amax reset (+ reciprocal of a given scale) and, for current scaling, the amax pass: shared with the FP8 casts
tweo_status_t launch_amax_prologue(const uint16_t* x, int64_t n, float* amax, uint32_t* sat_count, const float* scale_in,
                                   float* scale_inv, cudaStream_t st);
}

namespace {

using namespace tweo_detail;

constexpr int kThreads = 256;
constexpr float kE2M1Max = 6.0f;

// Two binary32 values -> their E2M1 codes (lo in the low nibble of `code`) and the E4M3 codes of the
// rounded values (lo in the low byte of `carrier`).  The clamp comes first: fminf / fmaxf return the
// operand that is not a NaN, so a NaN becomes +6 whatever the converter's own NaN rule is, and the
// saturation does not depend on the converter either; -0 and values that round to zero keep their sign.
__device__ __forceinline__ void cvt_e2m1x2(float lo, float hi, uint32_t& code, uint32_t& carrier) {
  lo = fmaxf(fminf(lo, kE2M1Max), -kE2M1Max);
  hi = fmaxf(fminf(hi, kE2M1Max), -kE2M1Max);
  asm("{\n"
      ".reg .b8 t;\n"
      ".reg .b32 h;\n"
      ".reg .b16 c;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t, %2, %3;\n"
      "cvt.u32.u8 %0, t;\n"
      "cvt.rn.f16x2.e2m1x2 h, t;\n"
      "cvt.rn.satfinite.e4m3x2.f16x2 c, h;\n"
      "cvt.u32.u16 %1, c;\n"
      "}"
      : "=r"(code), "=r"(carrier)
      : "f"(hi), "f"(lo));
}

// one byte of two packed codes -> the two carrier bytes (low nibble in the low byte)
__device__ __forceinline__ uint32_t carrier_of_packed(uint32_t byte) {
  uint32_t carrier;
  asm("{\n"
      ".reg .b8 t;\n"
      ".reg .b32 h;\n"
      ".reg .b16 c;\n"
      "cvt.u8.u32 t, %1;\n"
      "cvt.rn.f16x2.e2m1x2 h, t;\n"
      "cvt.rn.satfinite.e4m3x2.f16x2 c, h;\n"
      "cvt.u32.u16 %0, c;\n"
      "}"
      : "=r"(carrier)
      : "r"(byte));
  return carrier;
}

__device__ __forceinline__ float e2m1_scale_from_amax(float amax) {
  float s = 1.0f;
  if (amax > 0.0f && amax < __int_as_float(0x7F800000)) {
    s = __fdiv_rn(kE2M1Max, amax);
    if (s > 3.402823466e38f) s = 3.402823466e38f;
  }
  return s;
}

// 16 elements per thread and pass: two 16-byte loads -> 8 bytes of packed codes and / or 16 carrier bytes.
// CURRENT mode reads *amax (finished by the kernel before) and derives the scale; GIVEN mode reads *scale
// and folds |x| into *amax while casting.
template <bool GIVEN, int U>
__global__ void __launch_bounds__(kThreads)
fp4_cast_kernel(const uint16_t* x, int64_t n, float* scale, float* scale_inv, float* amax, uint8_t* q4, uint8_t* q8) {
  chain_release();
  chain_wait();
  float s;
  if (GIVEN) {
    s = *scale;
  } else {
    s = e2m1_scale_from_amax(*amax);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      *scale = s;
      *scale_inv = __fdiv_rn(1.0f, s);
    }
  }
  const uint64_t ss = pack_f32x2(s, s);
  const int64_t n16 = n >> 4;
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  uint2* q4v = reinterpret_cast<uint2*>(q4);
  uint4* q8v = reinterpret_cast<uint4*>(q8);
  const int64_t stride = (int64_t)gridDim.x * kThreads * U;
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
      if (i < n16) {
        const uint32_t w[8] = {v[u][0].x, v[u][0].y, v[u][0].z, v[u][0].w, v[u][1].x, v[u][1].y, v[u][1].z, v[u][1].w};
        uint32_t code[8], car[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float lo, hi;
          unpack_f32x2(mul_f32x2(bf16x2_to_f32x2(w[j]), ss), lo, hi);  // each lane rounded once
          cvt_e2m1x2(lo, hi, code[j], car[j]);
          if (GIVEN) absmax_f32(m0, m1, w[j]);
        }
        if (q4)
          __stcs(q4v + i, make_uint2(code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24),
                                     code[4] | (code[5] << 8) | (code[6] << 16) | (code[7] << 24)));
        if (q8)
          __stcs(q8v + i, make_uint4(car[0] | (car[1] << 16), car[2] | (car[3] << 16), car[4] | (car[5] << 16),
                                     car[6] | (car[7] << 16)));
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {  // ragged tail: n % 16 elements, in pairs (the tail starts at an even index)
    for (int64_t i = n16 << 4; i < n; i += 2) {
      const uint32_t w0 = x[i], w1 = i + 1 < n ? (uint32_t)x[i + 1] : 0u;
      uint32_t code, car;
      cvt_e2m1x2(__fmul_rn(bf16lo_to_f32(w0), s), __fmul_rn(bf16lo_to_f32(w1), s), code, car);
      if (i + 1 >= n) code &= 0x0Fu;  // an odd count leaves the last high nibble zero
      if (q4) q4[i >> 1] = (uint8_t)code;
      if (q8) {
        q8[i] = (uint8_t)(car & 0xFFu);
        if (i + 1 < n) q8[i + 1] = (uint8_t)(car >> 8);
      }
      if (GIVEN) absmax_f32(m0, m1, w0 | (w1 << 16));
    }
  }
  if (GIVEN) {
    uint32_t m = absmax_f32_bits(m0, m1);
    __shared__ uint32_t part[kThreads / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
      for (int w = 1; w < kThreads / 32; ++w) m = max(m, part[w]);
      if (m) atomicMax(reinterpret_cast<unsigned int*>(amax), m << 16);
    }
  }
}

// packed codes -> carriers: two 16-byte loads in flight per thread, 32 carrier bytes written for each
__global__ void __launch_bounds__(kThreads) fp4_unpack_kernel(const uint8_t* q4, int64_t n, uint8_t* q8) {
  chain_release();
  chain_wait();
  constexpr int U = 2;
  const int64_t n32 = n >> 5;
  const uint4* src = reinterpret_cast<const uint4*>(q4);
  uint4* dst = reinterpret_cast<uint4*>(q8);
  const int64_t stride = (int64_t)gridDim.x * kThreads * U;
  for (int64_t base = (int64_t)blockIdx.x * kThreads * U + threadIdx.x; base < n32; base += stride) {
    uint4 p[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t i = base + (int64_t)u * kThreads;
      if (i < n32) p[u] = __ldcs(src + i);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t i = base + (int64_t)u * kThreads;
      if (i >= n32) continue;
      const uint32_t w[4] = {p[u].x, p[u].y, p[u].z, p[u].w};
      uint32_t car[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) car[j] = carrier_of_packed((w[j >> 2] >> (8 * (j & 3))) & 0xFFu);
      __stcs(dst + 2 * i, make_uint4(car[0] | (car[1] << 16), car[2] | (car[3] << 16), car[4] | (car[5] << 16),
                                     car[6] | (car[7] << 16)));
      __stcs(dst + 2 * i + 1, make_uint4(car[8] | (car[9] << 16), car[10] | (car[11] << 16), car[12] | (car[13] << 16),
                                         car[14] | (car[15] << 16)));
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < 16) {  // ragged tail: n % 32 elements, one pair per thread
    const int64_t i = (n32 << 5) + 2 * threadIdx.x;
    if (i < n) {
      const uint32_t car = carrier_of_packed(q4[i >> 1]);
      q8[i] = (uint8_t)(car & 0xFFu);
      if (i + 1 < n) q8[i + 1] = (uint8_t)(car >> 8);
    }
  }
}

int cast_grid(int64_t n16, int u) {
  return balanced_grid((n16 + (int64_t)kThreads * u - 1) / ((int64_t)kThreads * u), (int64_t)sm_count() * 8);
}

}  // namespace

extern "C" tweo_status_t tweo_fp4_quantize(const uint16_t* x, int64_t n, int32_t mode, float* scale, float* scale_inv,
                                           float* amax, uint8_t* q4, uint8_t* q8, void* stream) {
  TWEO_LOG_CALL("tweo_fp4_quantize " "x=%p n=%lld mode=%d q4=%p q8=%p", (const void*)x,(long long)n,mode,(void*)q4,(void*)q8);
  if (n < 0 || !scale || !scale_inv || !amax) return TWEO_ERR_INVALID_ARG;
  if (mode != TWEO_SCALE_CURRENT && mode != TWEO_SCALE_GIVEN) return TWEO_ERR_INVALID_ARG;
  if (n > 0 && (!x || (!q4 && !q8))) return TWEO_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(q8) || (reinterpret_cast<uintptr_t>(q4) & 7u)) return TWEO_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  const bool given = mode == TWEO_SCALE_GIVEN;
  tweo_status_t ps = launch_amax_prologue(x, n, amax, nullptr, given ? (const float*)scale : (const float*)nullptr, scale_inv, st);
  if (ps != TWEO_OK) return ps;
  const int64_t n16 = n >> 4;
  const bool deep = n16 >= (int64_t)sm_count() * 8 * kThreads * 8;
  const dim3 grid(cast_grid(n16, deep ? 4 : 2));
  if (given) {
    if (deep) TWEO_CUDA_TRY(launch_chain(fp4_cast_kernel<true, 4>, grid, dim3(kThreads), 0, st, 0, x, n, scale, scale_inv, amax, q4, q8));
    else TWEO_CUDA_TRY(launch_chain(fp4_cast_kernel<true, 2>, grid, dim3(kThreads), 0, st, 0, x, n, scale, scale_inv, amax, q4, q8));
  } else {
    if (deep) TWEO_CUDA_TRY(launch_chain(fp4_cast_kernel<false, 4>, grid, dim3(kThreads), 0, st, 0, x, n, scale, scale_inv, amax, q4, q8));
    else TWEO_CUDA_TRY(launch_chain(fp4_cast_kernel<false, 2>, grid, dim3(kThreads), 0, st, 0, x, n, scale, scale_inv, amax, q4, q8));
  }
  count_launch();
  return check_launch("tweo_fp4_quantize");
}

extern "C" tweo_status_t tweo_fp4_unpack(const uint8_t* q4, int64_t n, uint8_t* q8, void* stream) {
  TWEO_LOG_CALL("tweo_fp4_unpack " "q4=%p n=%lld q8=%p", (const void*)q4,(long long)n,(void*)q8);
  if (n < 0 || (n > 0 && (!q4 || !q8))) return TWEO_ERR_INVALID_ARG;
  if (!aligned16(q8) || !aligned16(q4)) return TWEO_ERR_ALIGNMENT;
  if (n == 0) return TWEO_OK;
  cudaStream_t st = (cudaStream_t)stream;
  TWEO_CUDA_TRY(launch_chain(fp4_unpack_kernel, dim3(cast_grid(n >> 5, 2)), dim3(kThreads), 0, st, 0, q4, n, q8));
  count_launch();
  return check_launch("tweo_fp4_unpack");
}

extern "C" tweo_status_t tweo_w4a4_static_gemm(const uint16_t* x, int64_t ldx, const float* sx, const uint8_t* wq8,
                                               int64_t ldw, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                                               int64_t N, int64_t K, void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_w4a4_static_gemm " "M=%lld N=%lld K=%lld ldx=%lld ldw=%lld ws_bytes=%zu", (long long)M,(long long)N,(long long)K,(long long)ldx,(long long)ldw,ws_bytes);
  if (!x || !sx || !wq8 || !sw_inv || !y) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15) || ldx != K) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!ws || ws_bytes < tweo_workspace_bytes(TWEO_OP_W8A8, M, N, K)) return TWEO_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(ws) || !aligned16(x)) return TWEO_ERR_ALIGNMENT;
  float* scalars = reinterpret_cast<float*>(ws);  // [0] = 1 / sx, [1] = amax of x (by-product)
  uint8_t* carriers = reinterpret_cast<uint8_t*>(ws) + 256;
  tweo_status_t s = tweo_fp4_quantize(x, M * K, TWEO_SCALE_GIVEN, const_cast<float*>(sx), scalars, scalars + 1, nullptr,
                                      carriers, stream);
  if (s != TWEO_OK) return s;
  const size_t used = 256 + (((size_t)M * (size_t)K + 255) & ~(size_t)255);
  return gemm_fwd_codes(carriers, K, TWEO_E4M3, wq8, ldw, TWEO_E4M3, scalars, sw_inv, y, ldy, M, N, K, nullptr,
                        reinterpret_cast<char*>(ws) + used, ws_bytes - used, (cudaStream_t)stream, false);
}
