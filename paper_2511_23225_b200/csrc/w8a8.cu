// Static per-tensor W8A8 inference linear (E4M3 codes for weights and activations):
// optional saturating cast of bf16 activations with the calibrated scale, then the FP8
// forward GEMM with the dequantisation factor (1 / sx) * sw_inv.
#include "common.cuh"

namespace tweo_detail {
tweo_status_t gemm_fwd_codes(const uint8_t* xq, int64_t ldx, int fmt_x, const uint8_t* wq, int64_t ldw, int fmt_w,
                             const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                             int64_t N, int64_t K, const tweo_epilogue_t* epi, void* ws, size_t ws_bytes,
                             cudaStream_t st, bool sx_is_scale);
}

extern "C" tweo_status_t tweo_w8a8_static_gemm(const void* x, int32_t x_dtype, int64_t ldx, const float* sx,
                                               const uint8_t* wq, int64_t ldw, const float* sw_inv, uint16_t* y,
                                               int64_t ldy, int64_t M, int64_t N, int64_t K, void* ws,
                                               size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_w8a8_static_gemm " "M=%lld N=%lld K=%lld x_dtype=%d ldx=%lld ldw=%lld ws_bytes=%zu", (long long)M,(long long)N,(long long)K,x_dtype,(long long)ldx,(long long)ldw,ws_bytes);
  using namespace tweo_detail;
  if (!x || !sx || !wq || !sw_inv || !y) return TWEO_ERR_INVALID_ARG;
  if (x_dtype != TWEO_BF16 && x_dtype != TWEO_FP8_E4M3) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!ws || ws_bytes < tweo_workspace_bytes(TWEO_OP_W8A8, M, N, K)) return TWEO_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(ws) || !aligned16(x)) return TWEO_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  float* scalars = reinterpret_cast<float*>(ws);  // [0] = 1/sx, [1] = amax of x (by-product), [2] = scale_inv scratch
  const uint8_t* xq;
  int64_t ldxq;
  if (x_dtype == TWEO_BF16) {
    if (ldx != K) {
      // the cast runs over a dense tensor; a padded bf16 input would need a strided cast
      return TWEO_ERR_UNSUPPORTED_SHAPE;
    }
    uint8_t* codes = reinterpret_cast<uint8_t*>(ws) + 256;
    tweo_status_t s = tweo_quantize_per_tensor(reinterpret_cast<const uint16_t*>(x), M * K, TWEO_E4M3,
                                               TWEO_SCALE_GIVEN, const_cast<float*>(sx), scalars, scalars + 1,
                                               codes, nullptr, nullptr, 0, stream);
    if (s != TWEO_OK) return s;
    xq = codes;
    ldxq = K;
  } else {
    xq = reinterpret_cast<const uint8_t*>(x);   // the GEMM's epilogue forms 1 / *sx itself: no extra launch
    ldxq = ldx;
  }
  // what follows the scalars and the codes serves the GEMM's stream-K fix-up
  size_t used = 256;
  if (x_dtype == TWEO_BF16) used += ((size_t)M * (size_t)K + 255) & ~(size_t)255;
  const bool pre_cast = x_dtype != TWEO_BF16;
  return gemm_fwd_codes(xq, ldxq, TWEO_E4M3, wq, ldw, TWEO_E4M3, pre_cast ? sx : scalars, sw_inv, y, ldy, M, N, K, nullptr,
                        reinterpret_cast<char*>(ws) + used, ws_bytes - used, st, pre_cast);
}
