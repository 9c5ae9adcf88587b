// Several independent FP8 GEMMs in one launch of the CTA-pair kernel.  The case it was built for is
// the data gradient and the weight gradient of a linear layer, which the backward pass needs
// together and which share dY: launched separately, each leaves SMs idle -- the weight gradient of a
// transformer linear has only a few dozen (long) tiles, the data gradient often 1.3 waves of short
// ones.  More generally every launch pays a fixed cost (launch, set-up, the first cold loads, the
// last tile's epilogue: about 5 us, a third of a product of a GPT-2-small-sized linear), so up to
// kGroupMaxProblems products that do not depend on each other -- the forward products of several
// linears, or all their gradients -- share one.  The tiles of all products form one list, longest
// first, and the host assigns them to the CTA pairs by the longest-processing-time rule (each tile
// goes to the pair with the least work so far), so the long tiles start at once and the short ones
// fill in around them; one ramp-up and one tail for the whole group.
//
// The kernel is the CTA-pair kernel of gemm_pair.cuh (256 x 256 tiles, tcgen05 cta_group::2,
// TMA-fed ring, two accumulators in tensor memory, staged TMA-store epilogue) with the operand
// layouts taken at run time per product, bf16 outputs only and no splitting along the contraction.
// The QST instantiation also carries the fused epilogue of the training step per product: the maximum
// of |output| and the FP8 copy of the output with a given scale, staged in shared memory and stored by
// TMA like the bf16 tile (one operand stage less).  Every wait is bounded.
#pragma once

#include <cuda.h>

#include "gemm_common.cuh"
#include "tc_ptx.cuh"

namespace tweo_detail {

constexpr int kGroupMaxProblems = 8;
constexpr int kGroupListSmall = 2048;  // tile-list capacities the kernel is built for (the list travels in the
constexpr int kGroupListLarge = 8192;  // kernel parameters); beyond the large one tiles are dealt round-robin
constexpr int kGroupMaxPairs = 127;

struct GroupProblem {
  int32_t Md, Nd;
  int32_t tiles_m, tiles_n, k_blocks, raster_g;
  int32_t a_mn, b_mn;  // operand stored [Kc, rows] (1) or [rows, Kc] (0)
  uint32_t idesc;
  const float* sa_inv;
  const float* sb_inv;
  // fused epilogue (QST instantiation only)
  float* out_amax;        // nullptr: none
  const float* q_scale;   // nullptr: no FP8 copy
  int32_t q_fmt;
  int32_t pad;
};

template <int LIST>
struct alignas(64) PairGroupParams {
  CUtensorMap ma[kGroupMaxProblems], mb[kGroupMaxProblems], md[kGroupMaxProblems];
  CUtensorMap mq[kGroupMaxProblems];  // FP8 copies of the outputs (QST instantiation)
  GroupProblem pr[kGroupMaxProblems];
  int32_t n_problems;
  int32_t tile_start[kGroupMaxProblems + 1];  // product i owns the tile numbers [tile_start[i], tile_start[i + 1])
  int32_t total_tiles;
  int32_t use_lists;     // the per-pair lists are valid (total_tiles <= LIST)
  int32_t pad;
  uint16_t first[kGroupMaxPairs + 1];  // pair p computes list[first[p]] .. list[first[p + 1] - 1], in that order
  uint16_t list[LIST];                 // tile numbers
};

// The tile list of one CTA pair, identical in every warp role.
struct GroupSched {
  int pos, end, t, worker, workers;
  template <int LIST>
  __device__ GroupSched(const PairGroupParams<LIST>& g, int worker_, int workers_)
      : pos(g.use_lists ? g.first[worker_] : 0), end(g.use_lists ? g.first[worker_ + 1] : 0), t(-1), worker(worker_),
        workers(workers_) {}
  template <int LIST>
  __device__ bool next(const PairGroupParams<LIST>& g, int& prob, int& tile) {
    if (g.use_lists) {
      if (pos >= end) return false;
      t = g.list[pos++];
    } else {
      t = t < 0 ? worker : t + workers;
      if (t >= g.total_tiles) return false;
    }
    prob = 0;
    while (prob + 1 < g.n_problems && t >= g.tile_start[prob + 1]) ++prob;
    tile = t - g.tile_start[prob];
    return true;
  }
};

__device__ __forceinline__ void group_tile_coords(const GroupProblem& q, int tile, int& tm, int& tn) {
  const int per_band = q.raster_g * q.tiles_n;
  const int band = tile / per_band;
  const int first = band * q.raster_g;
  const int rows = min(q.raster_g, q.tiles_m - first);
  const int in = tile - band * per_band;
  tn = in / rows;
  tm = first + in - tn * rows;
}

// EPIW: epilogue warps per CTA (4 or 8; with 8, two warps share each quarter of the tensor-memory lanes and take
// half of a tile's columns each -- the fused epilogue of a short contraction is bound by the issue rate of one
// warp per scheduler).  EBUF: staging buffers per epilogue warp (2: a chunk is staged while the store of the
// one before it drains; 1: half the staging memory, which buys an operand stage).
template <int STAGES, int LIST, bool QST = false, int EPIW = 4, int EBUF = 2>
__global__ void __launch_bounds__(64 + 32 * EPIW, 1)
gemm_fp8_pair_group_kernel(const __grid_constant__ PairGroupParams<LIST> g) {
  constexpr int BN = 256;                 // tile columns of the pair
  constexpr uint32_t A_BYTES = BM * BK;   // this CTA's 128 rows of A
  constexpr uint32_t B_BYTES = 128 * BK;  // this CTA's 128 of the 256 columns of B
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr int CH = 64;                  // bf16 columns per 128-byte staging row

  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  constexpr uint32_t EPI_BUF = 32 * 128;
  static_assert(EPIW == 4 || EPIW == 8, "epilogue warps per CTA");
  static_assert(EBUF == 1 || EBUF == 2, "staging buffers per epilogue warp");
  constexpr uint32_t EPI_BYTES = EPIW * EBUF * EPI_BUF;
  constexpr uint32_t Q_BUF = 32 * 64;  // 32 rows x 64 one-byte codes
  constexpr uint32_t Q_BYTES = QST ? EPIW * EBUF * Q_BUF : 0;
  uint8_t* epi_smem = smem + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_smem + EPI_BYTES + Q_BYTES);
  // bars: [0,STAGES) full, [STAGES,2*STAGES) empty, then tfull[2], tempty[2]
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
  // Barriers and tensor memory are set up: the next kernel of the launch chain may start its own set-up.  Every
  // role prepares its tile list first and only then waits for the kernel before this one; nothing before
  // chain_wait() touches global memory.
  chain_release();

  const int pair = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      GroupSched sched(g, pair, num_pairs);
      for (int i = 0; i < g.n_problems; ++i) {
        tma_prefetch_desc(&g.ma[i]);
        tma_prefetch_desc(&g.mb[i]);
      }
      chain_wait();
      int prob, tile;
      while (ok && sched.next(g, prob, tile)) {
        const GroupProblem& q = g.pr[prob];
        int tm, tn;
        group_tile_coords(q, tile, tm, tn);
        const int m0 = tm * (2 * BM) + (int)rank * BM;  // this CTA's rows
        const int n0 = tn * BN + (int)rank * 128;       // this CTA's half of B
        const bool a_mn = q.a_mn != 0, b_mn = q.b_mn != 0;
        const CUtensorMap* ma = &g.ma[prob];
        const CUtensorMap* mb = &g.mb[prob];
        for (int kb = 0; kb < q.k_blocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          const int k0 = kb * BK;
          if (a_mn) tma_load_2d_pair(sa, ma, m0, k0, fb);
          else tma_load_2d_pair(sa, ma, k0, m0, fb);
          if (b_mn) tma_load_2d_pair(sb, mb, n0, k0, fb);
          else tma_load_2d_pair(sb, mb, k0, n0, fb);
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
      GroupSched sched(g, pair, num_pairs);
      chain_wait();
      int prob, tile;
      while (ok && sched.next(g, prob, tile)) {
        const GroupProblem& q = g.pr[prob];
        // K-major: step 32 bytes inside the swizzle span; MN-major: step 32 rows of 128 B
        const uint32_t a_step = q.a_mn ? UMMA_K * 128 : UMMA_K;
        const uint32_t b_step = q.b_mn ? UMMA_K * 128 : UMMA_K;
        const uint32_t idesc = q.idesc;
        const int k_blocks = q.k_blocks;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_f8_pair(d_tmem, make_smem_desc(sa + k * a_step, BK * 128), make_smem_desc(sb + k * b_step, BK * 128),
                         idesc, (uint32_t)((kb | k) != 0));
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
    // ------------------------------------------------------------ epilogue (warps 2.., both CTAs)
    chain_wait();
    const int quarter = warp & 3;  // the tensor-memory lanes a warp may read: (warp index mod 4) * 32 ...
    const uint32_t epi_base = smem_u32(epi_smem) + (uint32_t)(warp - 2) * (uint32_t)EBUF * EPI_BUF;
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t swz = (uint32_t)(lane & 7);
    const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
    const uint32_t q_base = smem_u32(epi_smem) + EPI_BYTES + (uint32_t)(warp - 2) * (uint32_t)EBUF * Q_BUF;
    // with 8 epilogue warps, warps 2-5 take the first half of a tile's chunks and warps 6-9 the second
    constexpr int NC_W = (BN / CH) / (EPIW / 4);
    const int c_first = ((warp - 2) >> 2) * NC_W;
    uint32_t it = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    // fused amax: the running maximum of |accumulator| of the product this warp is working on; written out
    // (scaled and rounded like the stored values) when the list moves on to another product and at the end
    float run_max = 0.0f, max_alpha = 0.0f;
    float* max_dst = nullptr;
    auto flush_max = [&]() {
      if (QST && max_dst) {
        float m = __uint_as_float(f32_to_bf16_bits(__fmul_rn(run_max, fabsf(max_alpha))) << 16);
        m = warp_max(m);
        if (lane == 0 && m > 0.0f) atomicMax(reinterpret_cast<unsigned int*>(max_dst), __float_as_uint(m));
      }
      run_max = 0.0f;
    };
    GroupSched sched(g, pair, num_pairs);
    int prob, tile;
    while (ok && sched.next(g, prob, tile)) {
      const GroupProblem& q = g.pr[prob];
      const CUtensorMap* md = &g.md[prob];
      const float alpha = __fmul_rn(__ldg(q.sa_inv), __ldg(q.sb_inv));
      const int Md = q.Md, Nd = q.Nd;
      float qs = 0.0f;
      if (QST) {
        if (q.out_amax != max_dst) {
          flush_max();
          max_dst = q.out_amax;
        }
        max_alpha = alpha;
        if (q.q_scale) qs = __ldg(q.q_scale);
      }
      int tm, tn;
      group_tile_coords(q, tile, tm, tn);
      const int m0 = tm * (2 * BM) + (int)rank * BM;
      const int n0 = tn * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row0 = m0 + quarter * 32;
#pragma unroll 1
      for (int c = c_first; c < c_first + NC_W; ++c) {
        const int col0 = n0 + c * CH;
        if (col0 >= Nd) break;
        uint32_t r[CH];
        const uint32_t taddr = tmem_base + tlane + (uint32_t)(acc * BN + c * CH);
        tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
        tmem_ld_wait();
        if (row0 >= Md) continue;
        const uint32_t ebuf = EBUF == 2 ? (it & 1u) : 0u;
        const uint32_t buf = epi_base + ebuf * EPI_BUF;
        if (lane == 0) bulk_wait_read<EBUF - 1>();
        __syncwarp();
        if (QST && max_dst) {
          // rows and columns beyond the output hold exact zeros (the loads fill them), so they do not count
#pragma unroll
          for (int j = 0; j < CH; ++j) run_max = fmaxf(run_max, fabsf(__uint_as_float(r[j])));
        }
        uint32_t packed[CH / 2];
#pragma unroll
        for (int j = 0; j < CH / 2; ++j)
          packed[j] = f32x2_to_bf16x2(__fmul_rn(__uint_as_float(r[2 * j]), alpha),
                                      __fmul_rn(__uint_as_float(r[2 * j + 1]), alpha));
#pragma unroll
        for (int j = 0; j < 8; ++j)
          st_shared_v4(buf + row_off + (((uint32_t)j ^ swz) << 4), packed[4 * j], packed[4 * j + 1], packed[4 * j + 2],
                       packed[4 * j + 3]);
        const uint32_t qbuf = q_base + ebuf * Q_BUF;
        if (QST && q.q_scale) {
          // 64 codes per row -> 32 rows x 64 B, 16-byte pieces XOR-swizzled with row bits 1-2
          const uint32_t qrow = qbuf + (uint32_t)lane * 64u;
          const uint32_t qswz = ((uint32_t)lane >> 1) & 3u;
#pragma unroll
          for (int g4 = 0; g4 < 4; ++g4) {
            uint32_t qq[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t w0 = packed[8 * g4 + 2 * j], w1 = packed[8 * g4 + 2 * j + 1];
              qq[j] = q.q_fmt == TWEO_E4M3 ? quant_words<TWEO_E4M3>(w0, w1, qs) : quant_words<TWEO_E5M2>(w0, w1, qs);
            }
            st_shared_v4(qrow + (((uint32_t)g4 ^ qswz) << 4), qq[0], qq[1], qq[2], qq[3]);
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(md, col0, row0, buf);
          if (QST && q.q_scale) tma_store_2d(&g.mq[prob], col0, row0, qbuf);
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
    flush_max();
    if (lane == 0) bulk_wait_all();
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
