// Tiles split along the contraction, shared by the single-CTA and the CTA-pair GEMM kernels.
//
// A worker (a CTA, or a CTA pair) whose share of the work covers only part of a tile's k-blocks
// does not finish that tile itself.  Each of its epilogue warps parks its 32 x BN block of the
// raw fp32 accumulator in the workspace ([column][row], so every store is one full line), hands
// the accumulator back to the MMA warp and takes a ticket on a counter of (tile, CTA of the pair,
// warp).  The warp that draws the LAST ticket of the tile adds the parked blocks of ALL shares in
// share order (= ascending k, whoever arrived last, so the sum does not depend on timing), runs
// the epilogue and resets the counter to zero.  Nobody waits for anybody, so the scheme needs no
// co-residency of the workers, holds across CUDA-graph replays (no launch-varying value is baked
// into the kernel parameters) and leaves the workspace ready for the next launch.
//
// Every worker parks at most two shares per launch: one that ends a tile (it starts in the middle,
// slot 0) and one that starts a tile (it ends in the middle, slot 1); a share in the middle of a
// tile is a worker's whole range and takes slot 0.
#pragma once

#include <cuda.h>

#include "gemm_common.cuh"
#include "tc_ptx.cuh"

namespace tweo_detail {

// BN: accumulator columns.  PAIR: the worker is a CTA pair (rank = CTA of the pair, the accumulator
// is returned through the leader's cluster barrier); otherwise a single CTA (rank 0, local barrier).
// Returns the maximum |bf16 output| this warp stored (0 if it was not the last share, or no amax wanted).
template <int BN, bool OUT_F32, bool PAIR>
__device__ __noinline__ float partial_share(const GemmParams& p, const CUtensorMap* tmap_d, int tile, int kb0,
                                            int worker, int num_workers, int rank, int wslot, uint32_t tacc,
                                            uint32_t tempty, float alpha, float qs, uint32_t epi_base, uint32_t it,
                                            int lane, int row0, int n0) {
  constexpr int CH = OUT_F32 ? 32 : 64;
  constexpr uint32_t EPI_BUF = 32 * 128;
  constexpr int CTAS = PAIR ? 2 : 1;
  constexpr size_t kCtaFloats = (size_t)128 * BN;   // one CTA's parked accumulator
  constexpr size_t kWarpFloats = (size_t)32 * BN;   // one epilogue warp's block of it
  float run_amax = 0.0f;
  float* slot = p.sk_partials + ((size_t)(worker * 2 + (kb0 > 0 ? 0 : 1)) * CTAS + rank) * kCtaFloats +
                (size_t)wslot * kWarpFloats;
#pragma unroll 1
  for (int g = 0; g < BN / 32; ++g) {
    uint32_t r[32];
    tmem_ld32(tacc + (uint32_t)(g * 32), r);
    tmem_ld_wait();
    float* dst = slot + g * 1024 + lane;
#pragma unroll
    for (int k = 0; k < 32; ++k) __stcg(dst + k * 32, __uint_as_float(r[k]));
  }
  tc_fence_before();
  __syncwarp();
  if (lane == 0) {
    if (PAIR) mbar_arrive_cluster(tempty);
    else mbar_arrive(tempty);
  }
  // which workers hold a share of this tile (they are consecutive)
  const int64_t t_begin = (int64_t)tile * p.k_blocks, t_end = t_begin + p.k_blocks;
  int j_first = worker;
  while (j_first > 0 && Sched::share_begin(p, j_first, num_workers) > t_begin) --j_first;
  int j_last = worker;
  while (j_last + 1 < num_workers && Sched::share_begin(p, j_last + 1, num_workers) < t_end) ++j_last;
  const int n_shares = j_last - j_first + 1;
  __threadfence();
  __syncwarp();
  uint32_t ticket = 0;
  uint32_t* counter = p.sk_counters + ((size_t)tile * CTAS + rank) * 4 + wslot;
  if (lane == 0) ticket = atomicAdd(counter, 1u);
  ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
  if (ticket + 1 != (uint32_t)n_shares) return 0.0f;  // not the last share of this tile: done
  __threadfence();
  if (lane == 0) *counter = 0u;  // ready for the next launch
  const uint32_t row_off = (uint32_t)lane * 128u;
  const uint32_t swz = (uint32_t)(lane & 7);
  const int row = row0 + lane;
#pragma unroll 1
  for (int c = 0; c < BN / CH; ++c) {
    const int col0 = n0 + c * CH;
    if (col0 >= p.Nd || row0 >= p.Md) break;  // uniform across the warp
    uint32_t r[CH];
#pragma unroll 1
    for (int sidx = 0; sidx < n_shares; ++sidx) {
      const int j = j_first + sidx;
      const int sel = Sched::share_begin(p, j, num_workers) > t_begin ? 0 : 1;
      const float* src = p.sk_partials + ((size_t)(j * 2 + sel) * CTAS + rank) * kCtaFloats +
                         (size_t)wslot * kWarpFloats + (size_t)(c * CH) * 32 + lane;
      if (sidx == 0) {
#pragma unroll
        for (int k = 0; k < CH; ++k) r[k] = __float_as_uint(__ldcg(src + k * 32));
      } else {
#pragma unroll
        for (int k = 0; k < CH; ++k) r[k] = __float_as_uint(__uint_as_float(r[k]) + __ldcg(src + k * 32));
      }
    }
    const uint32_t buf = epi_base + (it & 1u) * EPI_BUF;
    ++it;
    if (lane == 0) bulk_wait_read<1>();
    __syncwarp();
    if (OUT_F32) {
#pragma unroll
      for (int j = 0; j < 8; ++j)
        st_shared_v4(buf + row_off + (((uint32_t)j ^ swz) << 4),
                     __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j]), alpha)),
                     __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j + 1]), alpha)),
                     __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j + 2]), alpha)),
                     __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j + 3]), alpha)));
    } else {
      uint32_t packed[CH / 2];
#pragma unroll
      for (int j = 0; j < CH / 2; ++j)
        packed[j] = f32x2_to_bf16x2(__fmul_rn(__uint_as_float(r[2 * j]), alpha),
                                    __fmul_rn(__uint_as_float(r[2 * j + 1]), alpha));
#pragma unroll
      for (int j = 0; j < 8; ++j)
        st_shared_v4(buf + row_off + (((uint32_t)j ^ swz) << 4), packed[4 * j], packed[4 * j + 1], packed[4 * j + 2],
                     packed[4 * j + 3]);
      // fused amax / FP8 copy: single-CTA kernel only (the pair kernel's fused outputs take the staged route,
      // which never splits tiles)
      if (!PAIR && (p.out_amax || p.out_q) && row < p.Md) {
#pragma unroll 1
        for (int j = 0; j < CH / 4; ++j) {  // groups of four columns
          const uint32_t w0 = packed[2 * j], w1 = packed[2 * j + 1];
          float v[4] = {bf16lo_to_f32(w0), bf16hi_to_f32(w0), bf16lo_to_f32(w1), bf16hi_to_f32(w1)};
          if (col0 + 4 * j < p.Nd) {
            run_amax = fmaxf(run_amax, fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3]))));
            if (p.out_q) {
              const uint32_t q = p.q_fmt == TWEO_E4M3
                                     ? quant4<TWEO_E4M3>(__fmul_rn(v[0], qs), __fmul_rn(v[1], qs),
                                                         __fmul_rn(v[2], qs), __fmul_rn(v[3], qs))
                                     : quant4<TWEO_E5M2>(__fmul_rn(v[0], qs), __fmul_rn(v[1], qs),
                                                         __fmul_rn(v[2], qs), __fmul_rn(v[3], qs));
              *reinterpret_cast<uint32_t*>(p.out_q + (int64_t)row * p.ldq + col0 + 4 * j) = q;
            }
          }
        }
      }
    }
    fence_async_smem();
    __syncwarp();
    if (lane == 0) {
      if (OUT_F32 && p.accumulate) tma_reduce_add_2d(tmap_d, col0, row0, buf);
      else tma_store_2d(tmap_d, col0, row0, buf);
      bulk_commit();
    }
  }
  // the caller's buffer rotation does not know how many chunks were stored here
  if (lane == 0) bulk_wait_read<0>();
  __syncwarp();
  return run_amax;
}

}  // namespace tweo_detail
