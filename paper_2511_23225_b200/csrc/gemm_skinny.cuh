// Forward product for few tokens (M <= 128): Y[M,N] = Xq[M,K] . Wq[N,K]^T, the shape of a
// static W8A8 inference linear at small batch.  The work is streaming W once from HBM, so
// the kernel is organised around that: the operands are swapped -- 128 rows of W are the
// MMA's M dimension, the (padded) tokens its N dimension -- so the accumulator is only
// 128 x Mpad and nothing but W moves in bulk.  Each CTA takes one 128-row slab of W and one
// slice of K; slabs x slices is chosen to give every SM one CTA with a deep ring of TMA stages
// (up to 200 KB of loads in flight per SM).
//
// CTA = 192 threads: warp 0 issues TMA loads (W slab 128 x 128 B and X 'Mpad' x 128 B per
// k-block, 128-byte swizzle, rows beyond M zero-filled), warp 1 owns tensor memory and issues
// tcgen05.mma kind::f8f6f4 128 x Mpad x 32, warps 2-5 read the accumulator (lane = row of W =
// output column) and write Y.  With K sliced, every CTA parks its fp32 partial sums in the
// workspace ([column][token], a few KB), takes a ticket per (slab, warp), and the warp
// that draws the last ticket adds the slices in slice order and stores -- nobody waits, and
// the sum does not depend on timing.  All mbarrier waits are bounded.
#pragma once

#include <cuda.h>

#include "gemm_common.cuh"
#include "tc_ptx.cuh"

namespace tweo_detail {

constexpr int kSkinnyMaxStages = 11;

struct SkinnyParams {
  uint16_t* y;
  int64_t ldy;
  int32_t M, N, Mpad;      // Mpad: M rounded up to a multiple of 16 (<= 128)
  int32_t k_blocks;        // ceil(K / 128)
  int32_t slices;          // slices of K
  int32_t stages;          // TMA ring depth (<= kSkinnyMaxStages)
  uint32_t stage_bytes;    // 16 KB of W + Mpad * 128 B of X, rounded up to 1 KB
  uint32_t tmem_cols;      // power of two >= max(32, Mpad)
  uint32_t idesc;
  const float* sx_inv;
  const float* sw_inv;
  float* partials;         // [slab][slice][128 columns][Mpad] fp32, used when slices > 1
  uint32_t* counters;      // [slab][4] tickets, zero between launches
};

// 32 lanes x 16 consecutive 32-bit columns of tensor memory
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_fp8_skinny_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                       const __grid_constant__ SkinnyParams p) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * p.stage_bytes);
  // bars: [0,8) full, [8,16) empty, [16] accumulator complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kSkinnyMaxStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kSkinnyMaxStages + s); };
  const uint32_t done_bar = bar_base + 8u * (2 * kSkinnyMaxStages);

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(done_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int slab = blockIdx.x / p.slices;
  const int slice = blockIdx.x - slab * p.slices;
  const int n0 = slab * 128;
  const int kb0 = (int)((int64_t)p.k_blocks * slice / p.slices);
  const int kb1 = (int)((int64_t)p.k_blocks * (slice + 1) / p.slices);
  const uint32_t x_bytes = (uint32_t)p.Mpad * 128u;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) break;
        const uint32_t fb = full_bar(stage);
        mbar_expect_tx(fb, BM * BK + x_bytes);
        const uint32_t sw = smem_base + stage * p.stage_bytes;
        tma_load_2d(sw, &tmap_w, kb * BK, n0, fb);
        tma_load_2d(sw + BM * BK, &tmap_x, kb * BK, 0, fb);
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sw = smem_base + stage * p.stage_bytes;
        const uint32_t sx = sw + BM * BK;
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k)
          umma_f8(tmem_base, make_smem_desc(sw + k * UMMA_K, BK * 128), make_smem_desc(sx + k * UMMA_K, BK * 128),
                  p.idesc, (uint32_t)(kb != kb0 || k != 0));
        umma_commit(empty_bar(stage));
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
      if (ok) umma_commit(done_bar);
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;  // tensor-memory lanes [32*quarter, 32*quarter+32) belong to this warp
    const int col = n0 + quarter * 32 + lane;  // output column of this lane (= row of W)
    const float alpha = __fmul_rn(__ldg(p.sx_inv), __ldg(p.sw_inv));
    if (mbar_wait(done_bar, 0, abort_flag)) {
      tc_fence_after();
      const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16);
      if (p.slices == 1) {
        for (int c = 0; c < p.Mpad; c += 16) {
          uint32_t r[16];
          tmem_ld16(tacc + (uint32_t)c, r);
          tmem_ld_wait();
          if (col < p.N) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c + j < p.M)
                p.y[(int64_t)(c + j) * p.ldy + col] = (uint16_t)f32_to_bf16_bits(__fmul_rn(__uint_as_float(r[j]), alpha));
          }
        }
      } else {
        // park the partial sums: [column][token], a lane writes its column's tokens contiguously
        const size_t unit_floats = (size_t)128 * p.Mpad;
        float* mine = p.partials + (size_t)(slab * p.slices + slice) * unit_floats + (size_t)(quarter * 32 + lane) * p.Mpad;
        for (int c = 0; c < p.Mpad; c += 16) {
          uint32_t r[16];
          tmem_ld16(tacc + (uint32_t)c, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            __stcg(reinterpret_cast<float4*>(mine + c + j),
                   make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                               __uint_as_float(r[j + 3])));
        }
        __threadfence();
        __syncwarp();
        uint32_t ticket = 0;
        uint32_t* counter = p.counters + slab * 4 + quarter;
        if (lane == 0) ticket = atomicAdd(counter, 1u);
        ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
        if (ticket + 1 == (uint32_t)p.slices) {  // the last slice of this slab: add all slices in order
          __threadfence();
          if (lane == 0) *counter = 0u;  // ready for the next launch
          const float* base = p.partials + (size_t)slab * p.slices * unit_floats + (size_t)(quarter * 32 + lane) * p.Mpad;
          // 16 tokens of this column at a time, the loads of eight slices in flight together
          // (32 independent 16-byte loads); the additions still run in slice order
          for (int m = 0; m < p.M; m += 16) {
            float4 acc[4];
#pragma unroll 1
            for (int s0 = 0; s0 < p.slices; s0 += 8) {
              float4 v[8][4];
#pragma unroll
              for (int t = 0; t < 8; ++t) {
                const float4* src = reinterpret_cast<const float4*>(base + (size_t)(s0 + t) * unit_floats + m);
#pragma unroll
                for (int j = 0; j < 4; ++j) v[t][j] = (s0 + t < p.slices) ? __ldcg(src + j) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
#pragma unroll
              for (int t = 0; t < 8; ++t) {
                if (s0 + t < p.slices) {
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    if (s0 + t == 0) acc[j] = v[t][j];
                    else acc[j] = make_float4(acc[j].x + v[t][j].x, acc[j].y + v[t][j].y, acc[j].z + v[t][j].z,
                                              acc[j].w + v[t][j].w);
                  }
                }
              }
            }
            if (col < p.N) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float a4[4] = {acc[j].x, acc[j].y, acc[j].z, acc[j].w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (m + 4 * j + e < p.M)
                    p.y[(int64_t)(m + 4 * j + e) * p.ldy + col] = (uint16_t)f32_to_bf16_bits(__fmul_rn(a4[e], alpha));
              }
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

}  // namespace tweo_detail
