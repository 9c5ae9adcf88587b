// Forward product for few tokens (M <= 128): Y[M,N] = Xq[M,K] . Wq[N,K]^T, the shape of a
// static W8A8 inference linear at small batch.  The work is streaming W once from HBM, so
// the kernel is organised around that: the operands are swapped -- 128 rows of W are the
// MMA's M dimension, the (padded) tokens its N dimension -- so the accumulator is only
// 128 x Mpad and nothing but W moves in bulk.  Each CTA takes one 128-row slab of W and one
// slice of K; slabs x slices is chosen to give every SM one or two CTAs, each with a ring of TMA stages of
// up to 100 KB (two CTAs fit an SM, so in a launch chain the next kernel's CTAs fetch their first ring of W
// while this kernel's still reduce and write).
//
// CTA = 192 threads: warp 0 issues TMA loads (W slab 128 x 128 B and X 'Mpad' x 128 B per
// k-block, 128-byte swizzle, rows beyond M zero-filled), warp 1 owns tensor memory and issues
// tcgen05.mma kind::f8f6f4 128 x Mpad x 32, warps 2-5 read the accumulator (lane = row of W =
// output column) and write Y.  With K sliced, the slices of one slab form a thread-block cluster:
// every CTA parks its fp32 partial sums in its own shared memory ([token][128 columns], in the
// ring the loads no longer need), the cluster synchronises, and CTA r sums tokens r, r + S, ...
// over all S slices in slice order through distributed shared memory and writes those rows of Y
// (64 contiguous bytes per warp).  No workspace, no atomics, and the sum does not depend on
// timing.  All mbarrier waits are bounded; the cluster barrier is reached by every thread.
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
  int32_t slices;          // slices of K = CTAs per cluster (1, 2, 4 or 8)
  int32_t stages;          // TMA ring depth (<= kSkinnyMaxStages)
  uint32_t stage_bytes;    // 16 KB of W + Mpad * 128 B of X, rounded up to 1 KB
  uint32_t w_tx_bytes;     // bytes one W load reports to its barrier: the 16 KB it writes, or 8 KB for packed 4-bit
                           // codes (the load counts the bytes it fetched, not the padded groups it writes)
  uint32_t tmem_cols;      // power of two >= max(32, Mpad)
  uint32_t idesc;
  const float* sx_inv;
  const float* sw_inv;
  int32_t sx_is_scale;     // *sx_inv holds the activation scale itself, not its reciprocal
  // integer (Eq. 4) operands: y = float(acc) * (row_scale[token or 0] * post_scale) * col_scale[column or 0]
  const float* row_scale;
  const float* col_scale;
  int32_t row_scale_per_row, col_scale_per_col;
  float post_scale;
};

__device__ __forceinline__ uint32_t ld_shared_cluster_b32(uint32_t cluster_addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.b32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
  return v;
}

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

// One output value from an accumulator word: FP8 operands -- the binary32 sum times the dequantisation factor
// `alpha`; integer operands -- the int32 sum as binary32, times the token's scale (with Q_b^-2 folded in), times
// the column's scale `alpha` (the order the CTA-pair kernel's integer epilogue uses).
template <bool I8>
__device__ __forceinline__ float skinny_out(const SkinnyParams& p, uint32_t acc, int token, float alpha) {
  if (!I8) return __fmul_rn(__uint_as_float(acc), alpha);
  const float ar = __fmul_rn(__ldg(p.row_scale + (p.row_scale_per_row ? token : 0)), p.post_scale);
  return __fmul_rn(__fmul_rn(__int2float_rn((int)acc), ar), alpha);
}

// The cluster's reduction for one output column (this thread's): CTA `slice` of the cluster sums tokens slice,
// slice + S, ... over all S slices in slice order, reading the partial sums the CTAs parked in their shared memory
// ([token][128 columns] fp32) through distributed shared memory, TOK tokens at a time (TOK * SL loads in flight).
// SL: the slice count rounded up to 2, 4 or 8.
template <bool I8, int TOK, int SL>
__device__ __forceinline__ void skinny_reduce(const SkinnyParams& p, uint32_t mine, int slice, int n, float alpha) {
  uint32_t peer[SL];
#pragma unroll
  for (int sl = 0; sl < SL; ++sl) peer[sl] = map_to_cta(mine, (uint32_t)(sl < p.slices ? sl : 0));
  for (int t0 = slice; t0 < p.M; t0 += TOK * p.slices) {
    uint32_t v[TOK][SL];
#pragma unroll
    for (int u = 0; u < TOK; ++u) {
      const int t = t0 + u * p.slices;
#pragma unroll
      for (int sl = 0; sl < SL; ++sl)
        v[u][sl] = (sl < p.slices && t < p.M) ? ld_shared_cluster_b32(peer[sl] + (uint32_t)t * 512u) : 0u;
    }
#pragma unroll
    for (int u = 0; u < TOK; ++u) {
      const int t = t0 + u * p.slices;
      uint32_t acc;
      if (I8) {
        int a = (int)v[u][0];
#pragma unroll
        for (int sl = 1; sl < SL; ++sl)
          if (sl < p.slices) a += (int)v[u][sl];   // exact
        acc = (uint32_t)a;
      } else {
        float a = __uint_as_float(v[u][0]);
#pragma unroll
        for (int sl = 1; sl < SL; ++sl)
          if (sl < p.slices) a += __uint_as_float(v[u][sl]);  // slice order
        acc = __float_as_uint(a);
      }
      if (t < p.M && n < p.N) p.y[(int64_t)t * p.ldy + n] = (uint16_t)f32_to_bf16_bits(skinny_out<I8>(p, acc, t, alpha));
    }
  }
}

// I8: signed 8-bit operands (tcgen05 kind::i8, int32 accumulators: partial sums of K slices add exactly) with the
// Eq. 4 dequantisation in the epilogue, per tensor or per token (activation rows) / per channel (weight rows).
template <bool I8>
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

  // The kernel may have been launched while the kernel before it on the stream is still running (programmatic
  // dependent launch).  W is a static weight, not something that kernel produced, so the first ring of W loads is
  // issued at once; everything that can depend on the previous kernel -- the activations, the two scales, the
  // output buffer -- is touched only after chain_wait().
  chain_release();
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const int pre = min(p.stages, kb1 - kb0);   // the ring is empty: these stages need no wait
      for (int i = 0; i < pre; ++i) {
        mbar_expect_tx(full_bar(i), p.w_tx_bytes + x_bytes);
        tma_load_2d(smem_base + i * p.stage_bytes, &tmap_w, (kb0 + i) * BK, n0, full_bar(i));
      }
      chain_wait();
      for (int i = 0; i < pre; ++i)
        tma_load_2d(smem_base + i * p.stage_bytes + BM * BK, &tmap_x, (kb0 + i) * BK, 0, full_bar(i));
      int stage = pre == p.stages ? 0 : pre;
      uint32_t phase = pre == p.stages ? 1u : 0u;
      for (int kb = kb0 + pre; kb < kb1; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) break;
        const uint32_t fb = full_bar(stage);
        mbar_expect_tx(fb, p.w_tx_bytes + x_bytes);
        const uint32_t sw = smem_base + stage * p.stage_bytes;
        tma_load_2d(sw, &tmap_w, kb * BK, n0, fb);
        tma_load_2d(sw + BM * BK, &tmap_x, kb * BK, 0, fb);
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    chain_wait();
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
        for (int k = 0; k < BK / UMMA_K; ++k) {
          const uint64_t adesc = make_smem_desc(sw + k * UMMA_K, BK * 128), bdesc = make_smem_desc(sx + k * UMMA_K, BK * 128);
          if (I8) umma_i8(tmem_base, adesc, bdesc, p.idesc, (uint32_t)(kb != kb0 || k != 0));
          else umma_f8(tmem_base, adesc, bdesc, p.idesc, (uint32_t)(kb != kb0 || k != 0));
        }
        umma_commit(empty_bar(stage));
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
      if (ok) umma_commit(done_bar);
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    chain_wait();
    const int quarter = warp & 3;  // tensor-memory lanes [32*quarter, 32*quarter+32) belong to this warp
    const int col = n0 + quarter * 32 + lane;  // output column of this lane (= row of W)
    const float alpha = I8 ? __ldg(p.col_scale + (p.col_scale_per_col ? min(col, p.N - 1) : 0))
                           : dequant_alpha(p.sx_inv, p.sw_inv, p.sx_is_scale);
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
                p.y[(int64_t)(c + j) * p.ldy + col] = (uint16_t)f32_to_bf16_bits(skinny_out<I8>(p, r[j], c + j, alpha));
          }
        }
      } else {
        // park the partial sums in this CTA's shared memory: [token][128 columns] fp32 (the operand ring is
        // free: the accumulator-complete signal comes after the last MMA has read it)
        const uint32_t park = smem_base + (uint32_t)(quarter * 32 + lane) * 4u;
        for (int c = 0; c < p.Mpad; c += 16) {
          uint32_t r[16];
          tmem_ld16(tacc + (uint32_t)c, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j)
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(park + (uint32_t)(c + j) * 512u), "r"(r[j]) : "memory");
        }
      }
    }
  }

  if (p.slices > 1) {
    // every thread of every CTA of the cluster gets here, whatever happened above
    cluster_sync_all();  // all partial sums are parked and visible
    if (warp >= 2) {
      const int quarter = warp & 3;
      const int col = quarter * 32 + lane;
      const int n = n0 + col;
      const float alpha = I8 ? __ldg(p.col_scale + (p.col_scale_per_col ? min(n, p.N - 1) : 0))
                             : dequant_alpha(p.sx_inv, p.sw_inv, p.sx_is_scale);
      const uint32_t mine = smem_base + (uint32_t)col * 4u;
      // 64 remote loads in flight per thread whatever the slice count: 8, 16 or 32 tokens at a time
      if (p.slices > 4) skinny_reduce<I8, 8, 8>(p, mine, slice, n, alpha);
      else if (p.slices > 2) skinny_reduce<I8, 16, 4>(p, mine, slice, n, alpha);
      else skinny_reduce<I8, 32, 2>(p, mine, slice, n, alpha);
    }
    cluster_sync_all();  // nobody leaves while a peer may still read its shared memory
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

}  // namespace tweo_detail
