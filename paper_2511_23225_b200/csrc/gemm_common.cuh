// Definitions shared by the FP8 GEMM kernels: tile constants, the kernel parameter block, the
// workspace layout, the tile numbering and the work scheduler (whole tiles + tiles split along
// the contraction).  Not part of the public ABI.
#pragma once

#include <stdint.h>

#include "common.cuh"

namespace tweo_detail {

constexpr int BM = 128;      // rows of D per CTA tile = tcgen05 M per CTA (lanes of tensor memory)
constexpr int BK = 128;      // contraction bytes per stage = one 128-byte swizzle span
constexpr int UMMA_K = 32;   // contraction per instruction for 8-bit operands
constexpr int kThreads = 192;

struct GemmParams {
  void* d;
  int64_t ldd;
  int32_t Md, Nd, Kc;
  int32_t tiles_m, tiles_n, k_blocks;
  int32_t raster_g;    // tiles are numbered in bands of raster_g tile rows (see tile_coords)
  const float* sa_inv;
  const float* sb_inv;
  int32_t sa_is_scale;  // *sa_inv holds the scale itself, not its reciprocal (static W8A8: the calibrated scale)
  int32_t out_f32;     // 0: bf16 out, 1: fp32 out
  int32_t accumulate;  // fp32 out only
  float* out_amax;
  uint8_t* out_q;
  int64_t ldq;
  int32_t q_fmt;
  const float* q_scale;
  uint32_t idesc;
  // integer (Eq. 4) linear only: y = float(acc) * (row_scale[m or 0] * post_scale) * col_scale[n or 0]
  const float* row_scale;
  const float* col_scale;
  int32_t row_scale_per_row, col_scale_per_col;
  float post_scale;
  float q8_qmax;           // Q_b of an 8-bit (Eq. 4) output; its static scale is read from q_scale
  // stream-K: tiles [0, sk_tiles) are split along the contraction, the rest dealt whole
  int32_t sk_tiles;
  float* sk_partials;   // parked raw accumulators of the shares of split tiles: two slots per worker
  uint32_t* sk_counters;  // tickets per (tile, CTA of the pair, epilogue warp): [sk_tiles][2][4], single CTA [sk_tiles][4]
};

// Workspace layout of the linear calls (bytes from the workspace base):
//   [0, 4096)       unused
//   [4096, 12288)   ticket counters of the split tiles (CTA-pair kernel 8 words per tile, single-CTA kernel 4)
//   [12288, ...)    parked fp32 accumulators: 256 KB per SM
constexpr size_t kWsCountersOffset = 4096;
constexpr size_t kWsPartialsOffset = 12288;
constexpr size_t kWsPartialBytesPerSm = 256 * 1024;

// Tile index -> tile coordinates.  Tiles are numbered band by band: a band is raster_g tile
// rows high and is walked column by column, so the tiles in flight at any time cover a
// compact block (about raster_g rows x workers/raster_g columns) and the rows of A and the
// columns of B they share are re-read from L2 while they are still hot, instead of every wave
// sweeping all of A.
__device__ __forceinline__ void tile_coords(const GemmParams& p, int tile, int& tm, int& tn) {
  const int per_band = p.raster_g * p.tiles_n;
  const int band = tile / per_band;
  const int first = band * p.raster_g;
  const int rows = min(p.raster_g, p.tiles_m - first);
  const int in = tile - band * per_band;
  tn = in / rows;
  tm = first + in - tn * rows;
}

// The work list of one CTA, identical in the three roles (producer, MMA, epilogue).
struct Sched {
  int64_t u, u_end;   // stream-K units (tile * k_blocks + k-block) still to do
  int dp_tile, num_tiles, k_blocks, grid;
  __device__ Sched(const GemmParams& p, int cta, int grid_)
      : dp_tile(p.sk_tiles + cta), num_tiles(p.tiles_m * p.tiles_n), k_blocks(p.k_blocks), grid(grid_) {
    const int64_t total = (int64_t)p.sk_tiles * p.k_blocks;
    u = total * cta / grid_;
    u_end = total * (cta + 1) / grid_;
  }
  // first unit of CTA j's stream-K share
  __device__ static int64_t share_begin(const GemmParams& p, int j, int grid_) {
    return (int64_t)p.sk_tiles * p.k_blocks * j / grid_;
  }
  __device__ bool next(int& tile, int& kb0, int& kb1) {
    if (u < u_end) {
      tile = (int)(u / k_blocks);
      kb0 = (int)(u - (int64_t)tile * k_blocks);
      const int64_t len = min((int64_t)(k_blocks - kb0), u_end - u);
      kb1 = kb0 + (int)len;
      u += len;
      return true;
    }
    if (dp_tile < num_tiles) {
      tile = dp_tile;
      kb0 = 0;
      kb1 = k_blocks;
      dp_tile += grid;
      return true;
    }
    return false;
  }
};

// The tiles of one worker of the CTA-pair kernel, in the order all three warp roles walk them: the
// stream-K / round-robin list of Sched with the banded tile numbering.
struct TileWalk {
  Sched sched;
  __device__ TileWalk(const GemmParams& p, int worker, int workers) : sched(p, worker, workers) {}
  __device__ bool next(const GemmParams& p, int& tile, int& tm, int& tn, int& kb0, int& kb1) {
    if (!sched.next(tile, kb0, kb1)) return false;
    tile_coords(p, tile, tm, tn);
    return true;
  }
};

// ----------------------------------------------------------------- epilogue helpers
// Dequantisation factor of a product: (1 / scale_a) * (1 / scale_b), each reciprocal rounded once.
__device__ __forceinline__ float dequant_alpha(const float* sa, const float* sb_inv, int sa_is_scale) {
  float a = __ldg(sa);
  if (sa_is_scale) a = __fdiv_rn(1.0f, a);
  return __fmul_rn(a, __ldg(sb_inv));
}

template <int FMT>
__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d) {
  return cvt_fp8x2<FMT>(a, b) | (cvt_fp8x2<FMT>(c, d) << 16);
}

// Four bf16 values (two packed words) times the scale -> four FP8 codes.
template <int FMT>
__device__ __forceinline__ uint32_t quant_words(uint32_t w0, uint32_t w1, float qs) {
  return quant4<FMT>(__fmul_rn(bf16lo_to_f32(w0), qs), __fmul_rn(bf16hi_to_f32(w0), qs),
                     __fmul_rn(bf16lo_to_f32(w1), qs), __fmul_rn(bf16hi_to_f32(w1), qs));
}

// MLP activations of the forward epilogue (Sec. 3.2: GELU in the classic MLP, a gated unit in the
// Llama-style one), on binary32 values.
// 1: v * Phi(v).  Phi from the rational approximation of erfc by Hastings (Abramowitz & Stegun
//    7.1.26): erfc(x) = t (a1 + t (a2 + t (a3 + t (a4 + t a5)))) exp(-x^2), t = 1 / (1 + p x), x >= 0,
//    absolute error below 1.5e-7 -- three orders below the bf16 rounding that follows.
// 2: the tanh form with the hardware tanh (relative error 2^-11).
template <int ACT>
__device__ __forceinline__ float act_apply(float v) {
  if (ACT == 1) {
    const float x = fabsf(v) * 0.70710678118654752f;
    const float t = __fdividef(1.0f, fmaf(0.3275911f, x, 1.0f));
    float poly = fmaf(t, 1.061405429f, -1.453152027f);
    poly = fmaf(t, poly, 1.421413741f);
    poly = fmaf(t, poly, -0.284496736f);
    poly = fmaf(t, poly, 0.254829592f);
    const float half_erfc = 0.5f * t * poly * __expf(-x * x);   // Phi(-|v|)
    return v * (v >= 0.0f ? 1.0f - half_erfc : half_erfc);
  }
  if (ACT == 2) {
    const float u = 0.79788456080286536f * fmaf(0.044715f * v * v, v, v);
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
    const float h = 0.5f * v;
    return fmaf(h, t, h);
  }
  return v;
}
// SiLU(gate) * up = gate * up / (1 + exp(-gate))
__device__ __forceinline__ float swiglu(float gate, float up) {
  return __fdividef(gate, 1.0f + __expf(-gate)) * up;
}

}  // namespace tweo_detail
