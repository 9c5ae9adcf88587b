// CTA-pair FP8 GEMM kernel (included by the translation units that instantiate it).
// Two CTAs of a cluster (adjacent SMs) compute one 256 x 256 tile with tcgen05
// cta_group::2 instructions: each CTA stages its own 128 rows of A and only HALF of the
// B tile (128 of the 256 output columns), the pair's tensor cores read both halves, and
// each CTA's tensor memory receives the accumulator of its own 128 rows.  Per SM this
// moves 32 KB of operands per 128-deep contraction block instead of 48 KB, which is what
// lifts the kernel off the shared-memory fill limit.  Roles per CTA are those of the
// single-CTA kernel; only CTA 0 (the leader) issues MMAs.  Barriers:
//   full[s]    leader only : leader's producer arrives (+ expected bytes of BOTH CTAs' loads)
//   empty[s]   each CTA    : leader's MMA thread commits to its own and to the peer's
//   tfull[a]   each CTA    : same, once a tile's accumulator is complete
//   tempty[a]  leader only : the epilogue warps (4 or 8) of each CTA arrive (the peer's remotely; a relaxed
//                            arrival: a releasing one would wait for the warp's TMA stores to drain)
#pragma once

#include <cuda.h>

#include "gemm_common.cuh"
#include "gemm_split.cuh"
#include "tc_ptx.cuh"

namespace tweo_detail {

// I8: the operands are 8-bit integers (tcgen05 kind::i8, int32 accumulators) and the epilogue
// applies the Eq. 4 dequantisation with one scale per tensor or per row / column.
//
// ACT (forward product, bf16 / FP8 output): the MLP activation applied to the scaled accumulator
// before the one rounding to bf16 -- 1: GELU (erf), 2: GELU (tanh form), 3: SwiGLU.  For SwiGLU
// B holds the gate rows [0, Nd) followed by the up rows [Nd, 2 Nd): the leader CTA loads 128
// gate rows and its peer the matching 128 up rows, so accumulator columns [0,128) are the gate
// and [128,256) the up projection of the same 128 output columns, and the tile that is stored
// is 256 x 128: SiLU(gate) * up.  With p.d == nullptr only the FP8 copy / amax are produced.
//
// QST: the FP8 copy of the output leaves through shared memory and a TMA store (tmap_q: 64-byte
// rows, 64-byte swizzle) like the bf16 tile, instead of 16-byte stores from registers that touch
// 32 different rows per instruction.  Takes 16 KB of shared memory, so such kernels run with one
// stage less in the operand ring.
//
// EPIW: epilogue warps per CTA (4 or 8).  A warp reads the 32 tensor-memory lanes (warp index mod 4) allows
// it; with 8 warps two warps share each lane quarter and take half of the tile's columns each.  The
// epilogues that compute per element (activation, FP8 copy) are bound by the issue rate of one warp per
// scheduler at short contractions; a second warp per scheduler doubles it.  Costs 48 KB more staging memory
// (one operand stage less) and caps the kernel at 200 registers per thread.
//
// EBUF: staging buffers per epilogue warp (2: a chunk is staged while the store of the one before it drains;
// 1: half the staging memory, which buys an operand stage -- with eight warps the second warp of a scheduler
// covers the wait).
template <bool A_MN, bool B_MN, int STAGES, bool OUT_F32, bool I8 = false, int ACT = 0, bool QST = false, int EPIW = 4,
          int EBUF = 2>
__global__ void __launch_bounds__(64 + 32 * EPIW, 1)
gemm_fp8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_d, const __grid_constant__ CUtensorMap tmap_q,
                     const __grid_constant__ GemmParams p) {
  constexpr int BN = 256;                 // tile columns of the pair
  constexpr uint32_t A_BYTES = BM * BK;   // this CTA's 128 rows of A
  constexpr uint32_t B_BYTES = 128 * BK;  // this CTA's 128 of the 256 columns of B
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 512;

  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  constexpr uint32_t EPI_BUF = 32 * 128;
  constexpr uint32_t EPI_BYTES = EPIW * EBUF * EPI_BUF;
  static_assert(EBUF == 1 || EBUF == 2, "staging buffers per epilogue warp");
  static_assert(EPIW == 4 || EPIW == 8, "epilogue warps per CTA");
  constexpr bool Q8 = I8 && QST;                            // integer linear with an 8-bit (Eq. 4) output only
  constexpr uint32_t Q_BUF = 32 * 64;                       // 32 rows x 64 one-byte codes
  constexpr uint32_t Q_BYTES = QST ? EPIW * EBUF * Q_BUF : 0;
  uint8_t* epi_smem = smem + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_smem + EPI_BYTES + Q_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 2 * EPIW);  // the epilogue warps of both CTAs of the pair
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers are initialised before anyone signals across
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Barriers and tensor memory are set up.  The next kernel of the launch chain may start its own set-up now;
  // every role works out its tile list first and only then waits for the kernel before this one (whose
  // outputs may be this kernel's operands): nothing before chain_wait() touches global memory.
  chain_release();

  const int pair = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      TileWalk walk(p, pair, num_pairs);
      tma_prefetch_desc(&tmap_a);
      tma_prefetch_desc(&tmap_b);
      chain_wait();
      int tile, tm, tn, kb0, kb1;
      while (ok && walk.next(p, tile, tm, tn, kb0, kb1)) {
        const int m0 = tm * (2 * BM) + (int)rank * BM;  // this CTA's rows
        const int n0 = ACT == 3 ? tn * 128 + (int)rank * p.Nd  // gate rows (leader) / up rows (peer)
                                : tn * BN + (int)rank * 128;   // this CTA's half of B
        for (int kb = kb0; kb < kb1; ++kb) {
          const int k0 = kb * BK;
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          if (A_MN) tma_load_2d_pair(sa, &tmap_a, m0, k0, fb);
          else tma_load_2d_pair(sa, &tmap_a, k0, m0, fb);
          if (B_MN) tma_load_2d_pair(sb, &tmap_b, n0, k0, fb);
          else tma_load_2d_pair(sb, &tmap_b, k0, n0, fb);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && leader) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      TileWalk walk(p, pair, num_pairs);
      chain_wait();
      int tile, tm, tn, kb0, kb1;
      while (ok && walk.next(p, tile, tm, tn, kb0, kb1)) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = make_smem_desc(sa + (A_MN ? k * UMMA_K * 128 : k * UMMA_K), BK * 128);
            const uint64_t bdesc = make_smem_desc(sb + (B_MN ? k * UMMA_K * 128 : k * UMMA_K), BK * 128);
            if (I8) umma_i8_pair(d_tmem, adesc, bdesc, p.idesc, (uint32_t)(kb != kb0 || k != 0));
            else umma_f8_pair(d_tmem, adesc, bdesc, p.idesc, (uint32_t)(kb != kb0 || k != 0));
          }
          umma_commit_pair(map_to_cta(empty_bar(stage), 0));  // frees the stage in both CTAs
          umma_commit_pair(map_to_cta(empty_bar(stage), 1));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(map_to_cta(tfull_bar(acc), 0));      // accumulator complete, both CTAs
        umma_commit_pair(map_to_cta(tfull_bar(acc), 1));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2 .. 1 + EPIW, both CTAs)
    chain_wait();
    const int quarter = warp & 3;
    const float alpha = I8 ? 1.0f : dequant_alpha(p.sa_inv, p.sb_inv, p.sa_is_scale);
    const float qs = p.out_q ? (Q8 ? __fdiv_rn(p.q8_qmax, __ldg(p.q_scale)) : __ldg(p.q_scale)) : 0.0f;
    constexpr int CH = OUT_F32 ? 32 : 64;
    const uint32_t epi_base = smem_u32(epi_smem) + (uint32_t)(warp - 2) * (uint32_t)EBUF * EPI_BUF;
    const uint32_t q_base = smem_u32(epi_smem) + EPI_BYTES + (uint32_t)(warp - 2) * (uint32_t)EBUF * Q_BUF;
    // Running maximum for the fused amax.  Rounding to bf16 and the multiplication by the (positive) dequantisation
    // scale are monotone in the magnitude, so max |bf16(acc * alpha)| = bf16(max |acc| * alpha): without an activation
    // the maximum runs over the raw accumulators (one instruction per element), with one over the activation's
    // binary32 results; the scale and the rounding are applied once at the end.  Accumulator rows and columns beyond
    // the output are zero (the loader zero-fills), except the columns of a ragged SwiGLU tile, which are masked.
    float run_max = 0.0f;
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t swz = (uint32_t)(lane & 7);
    const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
    uint32_t it = 0;
    float run_amax = 0.0f;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    TileWalk walk(p, pair, num_pairs);
    int tile, tm, tn, kb0, kb1;
    while (ok && walk.next(p, tile, tm, tn, kb0, kb1)) {
      const int m0 = tm * (2 * BM) + (int)rank * BM;
      const int n0 = ACT == 3 ? tn * 128 : tn * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row0 = m0 + quarter * 32;
      const int row = row0 + lane;
      if (ACT == 0 && !QST && EBUF == 2 && (kb0 != 0 || kb1 != p.k_blocks)) {
        // part of a split tile: park the accumulator; the last share to arrive stores the tile
        const float part_amax = partial_share<BN, OUT_F32, true>(
            p, &tmap_d, tile, kb0, pair, num_pairs, (int)rank, warp - 2,
            tmem_base + tlane + (uint32_t)(acc * BN), map_to_cta(tempty_bar(acc), 0), alpha, qs, epi_base, it, lane,
            row0, n0);
        it += BN / CH;  // keeps the staging-buffer rotation in step whether or not this warp stored
        run_amax = fmaxf(run_amax, part_amax);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        continue;
      }
      // with 8 epilogue warps, warps 2-5 take the first half of the tile's chunks and warps 6-9 the second
      constexpr int NC = (ACT == 3 ? 128 : BN) / CH, NC_W = NC / (EPIW / 4);
      const int c_first = ((warp - 2) >> 2) * NC_W;
#pragma unroll 1
      for (int c = c_first; c < c_first + NC_W; ++c) {
        const int col0 = n0 + c * CH;
        if (col0 >= p.Nd) break;
        uint32_t r[CH];
        const uint32_t taddr = tmem_base + tlane + (uint32_t)(acc * BN + c * CH);
        tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        if (!OUT_F32) tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[CH - 32]));
        tmem_ld_wait();
        if (row0 >= p.Md) continue;
        if (ACT == 3) {
          // r holds 64 gate columns; fetch the matching up columns 32 at a time and combine in place
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t u[32];
            tmem_ld32(taddr + 128 + 32 * h, u);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j)
              r[32 * h + j] = __float_as_uint(swiglu(__fmul_rn(__uint_as_float(r[32 * h + j]), alpha),
                                                     __fmul_rn(__uint_as_float(u[j]), alpha)));
          }
        }
        if (I8) {
          // int32 accumulators -> binary32, then the two Eq. 4 scales (row first, then column)
          const float ar = __fmul_rn(__ldg(p.row_scale + (p.row_scale_per_row ? min(row, p.Md - 1) : 0)), p.post_scale);
          const float ac0 = __ldg(p.col_scale);
          if (p.col_scale_per_col && col0 + CH <= p.Nd && (reinterpret_cast<uintptr_t>(p.col_scale) & 15u) == 0) {
            // a whole chunk of per-channel scales: 16-byte loads (the same addresses in every lane)
            const float4* cs = reinterpret_cast<const float4*>(p.col_scale + col0);
#pragma unroll
            for (int j4 = 0; j4 < CH / 4; ++j4) {
              const float4 a4 = __ldg(cs + j4);
              r[4 * j4] = __float_as_uint(__fmul_rn(__fmul_rn(__int2float_rn((int)r[4 * j4]), ar), a4.x));
              r[4 * j4 + 1] = __float_as_uint(__fmul_rn(__fmul_rn(__int2float_rn((int)r[4 * j4 + 1]), ar), a4.y));
              r[4 * j4 + 2] = __float_as_uint(__fmul_rn(__fmul_rn(__int2float_rn((int)r[4 * j4 + 2]), ar), a4.z));
              r[4 * j4 + 3] = __float_as_uint(__fmul_rn(__fmul_rn(__int2float_rn((int)r[4 * j4 + 3]), ar), a4.w));
            }
          } else {
#pragma unroll
            for (int j = 0; j < CH; ++j) {
              const float ac = p.col_scale_per_col ? __ldg(p.col_scale + min(col0 + j, p.Nd - 1)) : ac0;
              r[j] = __float_as_uint(__fmul_rn(__fmul_rn(__int2float_rn((int)r[j]), ar), ac));
            }
          }
        }
        const uint32_t ebuf = EBUF == 2 ? (it & 1u) : 0u;
        const uint32_t buf = epi_base + ebuf * EPI_BUF;
        if (lane == 0) bulk_wait_read<EBUF - 1>();
        __syncwarp();
        if (Q8) {
          // Eq. 4 with the static output scale on the binary32 results: clamp(rne_int(y * (Q_b / s))), NaN -> 0
          const uint32_t qrow = q_base + ebuf * Q_BUF + (uint32_t)lane * 64u;
          const uint32_t qswz = ((uint32_t)lane >> 1) & 3u;
          const int qmax = (int)p.q8_qmax;
#pragma unroll
          for (int g4 = 0; g4 < 4; ++g4) {
            uint32_t q[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t w = 0u;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int c = max(-qmax, min(qmax, __float2int_rn(__fmul_rn(__uint_as_float(r[16 * g4 + 4 * j + e]), qs))));
                w |= ((uint32_t)c & 0xFFu) << (8 * e);
              }
              q[j] = w;
            }
            st_shared_v4(qrow + (((uint32_t)g4 ^ qswz) << 4), q[0], q[1], q[2], q[3]);
          }
        } else if (OUT_F32) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            st_shared_v4(buf + row_off + (((uint32_t)j ^ swz) << 4),
                         __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j]), alpha)),
                         __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j + 1]), alpha)),
                         __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j + 2]), alpha)),
                         __float_as_uint(__fmul_rn(__uint_as_float(r[4 * j + 3]), alpha)));
        } else {
          uint32_t packed[CH / 2];
          const bool want_max = QST && p.out_amax != nullptr;
          const bool whole = ACT != 3 || col0 + CH <= p.Nd;   // only a ragged SwiGLU chunk has live columns beyond Nd
          if (ACT == 0 && want_max) {
#pragma unroll
            for (int j = 0; j < CH; ++j) run_max = fmaxf(run_max, fabsf(__uint_as_float(r[j])));
          }
#pragma unroll
          for (int j = 0; j < CH / 2; ++j) {
            float v0, v1;
            if (ACT == 3) {
              v0 = __uint_as_float(r[2 * j]);
              v1 = __uint_as_float(r[2 * j + 1]);
            } else {
              v0 = act_apply<ACT>(__fmul_rn(__uint_as_float(r[2 * j]), alpha));
              v1 = act_apply<ACT>(__fmul_rn(__uint_as_float(r[2 * j + 1]), alpha));
            }
            if (ACT != 0 && want_max) {
              if (whole) {
                run_max = fmaxf(run_max, fmaxf(fabsf(v0), fabsf(v1)));
              } else {
                if (col0 + 2 * j < p.Nd) run_max = fmaxf(run_max, fabsf(v0));
                if (col0 + 2 * j + 1 < p.Nd) run_max = fmaxf(run_max, fabsf(v1));
              }
            }
            packed[j] = f32x2_to_bf16x2(v0, v1);
          }
          if (ACT == 0 || p.d != nullptr) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              st_shared_v4(buf + row_off + (((uint32_t)j ^ swz) << 4), packed[4 * j], packed[4 * j + 1],
                           packed[4 * j + 2], packed[4 * j + 3]);
          }
          if (QST) {
            if (p.out_q) {
              // 64 codes per row -> 32 rows x 64 B, 16-byte pieces XOR-swizzled with row bits 1-2
              const uint32_t qbuf = q_base + ebuf * Q_BUF;
              const uint32_t qrow = qbuf + (uint32_t)lane * 64u;
              const uint32_t qswz = ((uint32_t)lane >> 1) & 3u;
#pragma unroll
              for (int g4 = 0; g4 < 4; ++g4) {
                uint32_t q[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const uint32_t w0 = packed[8 * g4 + 2 * j], w1 = packed[8 * g4 + 2 * j + 1];
                  q[j] = p.q_fmt == TWEO_E4M3 ? quant_words<TWEO_E4M3>(w0, w1, qs) : quant_words<TWEO_E5M2>(w0, w1, qs);
                }
                st_shared_v4(qrow + (((uint32_t)g4 ^ qswz) << 4), q[0], q[1], q[2], q[3]);
              }
            }
          }
          // (without QST the kernel has no fused outputs: the host sends those products to a QST instantiation)
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (!Q8 && (ACT == 0 || p.d != nullptr)) {
            if (OUT_F32 && p.accumulate) tma_reduce_add_2d(&tmap_d, col0, row0, buf);
            else tma_store_2d(&tmap_d, col0, row0, buf);
          }
          if (QST && p.out_q) tma_store_2d(&tmap_q, col0, row0, q_base + ebuf * Q_BUF);
          bulk_commit();
        }
        ++it;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_relaxed(map_to_cta(tempty_bar(acc), 0));  // the leader's barrier
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (lane == 0) bulk_wait_all();
    if (p.out_amax) {
      if (QST) {
        const float m = ACT == 0 ? __fmul_rn(run_max, fabsf(alpha)) : run_max;
        run_amax = fmaxf(run_amax, __uint_as_float(f32_to_bf16_bits(m) << 16));   // the same rounding the stored values got
      }
      run_amax = warp_max(run_amax);
      if (lane == 0 && run_amax > 0.0f)
        atomicMax(reinterpret_cast<unsigned int*>(p.out_amax), __float_as_uint(run_amax));
    }
  }

  // Neither CTA may leave (or free tensor memory) while the other can still signal its
  // barriers or have MMAs reading its shared memory.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}


}  // namespace tweo_detail
