// FP8 x FP8 -> fp32 GEMMs of the linear layer (forward, data gradient, weight gradient)
// on the sm_100a tensor cores: tcgen05.mma kind::f8f6f4, operands staged in shared memory
// by TMA (128-byte swizzle), accumulators in tensor memory, epilogue through tcgen05.ld.
//
// One kernel serves all three products.  It computes D[Md,Nd] = A . B over a contraction
// of length Kc, where each operand is either
//   "K-major"  : stored [rows = Md or Nd, Kc] with the contraction contiguous, or
//   "MN-major" : stored [Kc, rows] with the output dimension contiguous.
//     forward  Y  = Xq  . Wq^T : A = Xq  [M,K]  K-major , B = Wq [N,K]  K-major , Kc = K
//     dgrad    dX = dYq . Wq   : A = dYq [M,N]  K-major , B = Wq [N,K]  MN-major, Kc = N
//     wgrad    dW = dYq^T . Xq : A = dYq [M,N]  MN-major, B = Xq [M,K]  MN-major, Kc = M
//   so no operand is ever transposed in memory: the major-ness bits of the instruction
//   descriptor and the shared-memory descriptors absorb the layout.
//
// CTA = 192 threads: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the
// MMAs (one thread), warps 2-5 are the epilogue (each reads its own 32-lane quarter of
// tensor memory, converts, stages 32 rows x 128 bytes in swizzled shared memory and hands
// them to a TMA store, so global writes are full lines and ragged edges are clipped by
// the hardware).  The kernel is persistent (grid = #SMs, static tile striding) with a
// ring of shared-memory stages and two accumulators in tensor memory, so the epilogue of
// tile i overlaps the main loop of tile i+1.
//
// Scheduling.  Tiles are dealt round-robin to the CTAs.  When that would leave SMs idle
// (fewer tiles than SMs, or a ragged last wave) and the contraction is long, the last
// tiles are instead cut along the contraction ("stream-K"): their (tile, k-block) units
// are split evenly over all CTAs.  Every share of such a tile parks its raw fp32 accumulator
// in a workspace slot and takes a ticket; the share that draws the tile's last ticket adds
// all of them in share order (fixed order => reproducible) and runs the epilogue
// (gemm_split.cuh).  No CTA waits for another one.
//
// Every mbarrier wait is bounded: on expiry the CTA records TWEO_ERR_TIMEOUT in
// a device status word, drains and exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <mutex>
#include <queue>
#include <utility>
#include <vector>

#include "common.cuh"

#include "gemm_common.cuh"
#include "gemm_pair.cuh"
#include "gemm_pair_group.cuh"
#include "gemm_skinny.cuh"
#include "gemm_split.cuh"
#include "tc_ptx.cuh"

namespace {

using namespace tweo_detail;

// ----------------------------------------------------------------- the kernel
template <int BN, bool A_MN, bool B_MN, int STAGES, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_fp8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                const __grid_constant__ CUtensorMap tmap_d, const GemmParams p) {
  constexpr uint32_t A_BYTES = BM * BK;
  constexpr uint32_t B_BYTES = BN * BK;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN >= 512 ? 512 : (2 * BN >= 256 ? 256 : (2 * BN >= 128 ? 128 : 64));
  static_assert(BN % 16 == 0 && BN >= 16 && BN <= 256, "tcgen05 N for M = 128");
  static_assert(!B_MN || BN % 128 == 0, "MN-major B tiles come in 128-wide slabs");

  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  // epilogue staging: per epilogue warp two buffers of 32 rows x 128 bytes (128-byte swizzle)
  constexpr uint32_t EPI_BUF = 32 * 128;
  constexpr uint32_t EPI_BYTES = 4 * 2 * EPI_BUF;
  uint8_t* epi_smem = smem + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_smem + EPI_BYTES);
  // bars: [0,STAGES) full, [STAGES,2*STAGES) empty, then tmem_full[2], tmem_empty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
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
      mbar_init(tempty_bar(a), 4);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      Sched sched(p, blockIdx.x, gridDim.x);
      int tile, kb0, kb1;
      while (ok && sched.next(tile, kb0, kb1)) {
        int tm, tn;
        tile_coords(p, tile, tm, tn);
        const int m0 = tm * BM;
        const int n0 = tn * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, STAGE_BYTES);
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          const int k0 = kb * BK;
          if (A_MN) tma_load_2d(sa, &tmap_a, m0, k0, fb);
          else tma_load_2d(sa, &tmap_a, k0, m0, fb);
          if (B_MN) {
#pragma unroll
            for (int j = 0; j < BN / 128; ++j) tma_load_2d(sb + j * (BK * 128), &tmap_b, n0 + j * 128, k0, fb);
          } else {
            tma_load_2d(sb, &tmap_b, k0, n0, fb);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      // Do not leave while copies may still be landing in this CTA's shared memory:
      // wait (bounded) for the last fill of every stage.  On the normal path these
      // phases completed long ago.
      if (!ok) {
        for (int s = 0; s < STAGES; ++s) {
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(full_bar(s), 0) && !mbar_try_wait(full_bar(s), 1)) {
            if (globaltimer_ns() - t0 > 100000000ull) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      Sched sched(p, blockIdx.x, gridDim.x);
      int tile, kb0, kb1;
      while (ok && sched.next(tile, kb0, kb1)) {
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
            // K-major: step 32 bytes inside the swizzle span; MN-major: step 32 rows of 128 B
            const uint64_t adesc = make_smem_desc(sa + (A_MN ? k * UMMA_K * 128 : k * UMMA_K), BK * 128);
            const uint64_t bdesc = make_smem_desc(sb + (B_MN ? k * UMMA_K * 128 : k * UMMA_K), BK * 128);
            umma_f8(d_tmem, adesc, bdesc, p.idesc, (uint32_t)(kb != kb0 || k != 0));
          }
          umma_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));      // accumulator complete -> epilogue
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;  // tensor-memory lanes [32*quarter, 32*quarter+32) belong to this warp
    const float alpha = dequant_alpha(p.sa_inv, p.sb_inv, p.sa_is_scale);
    const float qs = p.out_q ? __ldg(p.q_scale) : 0.0f;
    constexpr int CH = OUT_F32 ? 32 : 64;  // output columns per 128-byte staging row
    const uint32_t epi_base = smem_u32(epi_smem) + (uint32_t)(warp - 2) * 2u * EPI_BUF;
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t swz = (uint32_t)(lane & 7);
    uint32_t it = 0;
    float run_amax = 0.0f;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    Sched sched(p, blockIdx.x, gridDim.x);
    int tile, kb0, kb1;
    while (ok && sched.next(tile, kb0, kb1)) {
      int tm, tn;
      tile_coords(p, tile, tm, tn);
      const int m0 = tm * BM;
      const int n0 = tn * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
      if (kb0 != 0 || kb1 != p.k_blocks) {
        // part of a split tile: park the accumulator; the last share to arrive stores the tile
        const float part_amax = partial_share<BN, OUT_F32, false>(
            p, &tmap_d, tile, kb0, (int)blockIdx.x, (int)gridDim.x, 0, quarter,
            tmem_base + tlane + (uint32_t)(acc * BN), tempty_bar(acc), alpha, qs, epi_base, it, lane,
            m0 + quarter * 32, n0);
        it += BN / CH;  // keeps the staging-buffer rotation in step whether or not this warp stored
        run_amax = fmaxf(run_amax, part_amax);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        continue;
      }
      const int row0 = m0 + quarter * 32;
      const int row = row0 + lane;
      const bool row_ok = row < p.Md;
#pragma unroll 1
      for (int c = 0; c < BN / CH; ++c) {
        const int col0 = n0 + c * CH;
        if (col0 >= p.Nd) break;  // uniform across the warp
        uint32_t r[CH];
        const uint32_t taddr = tmem_base + tlane + (uint32_t)(acc * BN + c * CH);
        tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        if (!OUT_F32) tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[CH - 32]));
        tmem_ld_wait();
        if (row0 >= p.Md) continue;  // whole warp past the ragged edge (uniform)
        const uint32_t buf = epi_base + (it & 1u) * EPI_BUF;
        // the store issued two chunks ago must have finished reading this buffer
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
            st_shared_v4(buf + row_off + (((uint32_t)j ^ swz) << 4), packed[4 * j], packed[4 * j + 1],
                         packed[4 * j + 2], packed[4 * j + 3]);
          if ((p.out_amax || p.out_q) && row_ok) {
            // fused amax / cast act on the bf16-rounded values just staged
#pragma unroll
            for (int h = 0; h < 2; ++h) {  // two groups of 32 columns
              uint32_t q[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const uint32_t w0 = packed[16 * h + 2 * j], w1 = packed[16 * h + 2 * j + 1];
                float v[4] = {bf16lo_to_f32(w0), bf16hi_to_f32(w0), bf16lo_to_f32(w1), bf16hi_to_f32(w1)};
                if (col0 + 32 * h + 4 * j < p.Nd)
                  run_amax = fmaxf(run_amax, fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3]))));
                if (p.out_q) {
                  if (p.q_fmt == TWEO_E4M3)
                    q[j] = quant4<TWEO_E4M3>(__fmul_rn(v[0], qs), __fmul_rn(v[1], qs), __fmul_rn(v[2], qs),
                                             __fmul_rn(v[3], qs));
                  else
                    q[j] = quant4<TWEO_E5M2>(__fmul_rn(v[0], qs), __fmul_rn(v[1], qs), __fmul_rn(v[2], qs),
                                             __fmul_rn(v[3], qs));
                }
              }
              if (p.out_q) {
                uint8_t* qrow = p.out_q + (int64_t)row * p.ldq + col0 + 32 * h;
                if (col0 + 32 * h < p.Nd) *reinterpret_cast<uint4*>(qrow) = make_uint4(q[0], q[1], q[2], q[3]);
                if (col0 + 32 * h + 16 < p.Nd) *reinterpret_cast<uint4*>(qrow + 16) = make_uint4(q[4], q[5], q[6], q[7]);
              }
            }
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (OUT_F32 && p.accumulate) tma_reduce_add_2d(&tmap_d, col0, row0, buf);
          else tma_store_2d(&tmap_d, col0, row0, buf);
          bulk_commit();
        }
        ++it;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (lane == 0) bulk_wait_all();  // staged tiles must have left shared memory before the CTA exits
    if (p.out_amax) {
      run_amax = warp_max(run_amax);
      if (lane == 0 && run_amax > 0.0f)
        atomicMax(reinterpret_cast<unsigned int*>(p.out_amax), __float_as_uint(run_amax));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}


// Clears the amax cell of a fused epilogue.  Launched in the chain: the previous kernel may still read the cell.
__global__ void zero_float_kernel(float* p) {
  chain_release();
  chain_wait();
  *p = 0.0f;
}

// Self-test of the bounded wait: one thread waits on a barrier phase that nobody completes, with the
// given limit; the wait gives up, records the expiry in the status word and the kernel returns.
__global__ void bounded_wait_selftest_kernel(uint64_t limit_ns, unsigned int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait_limit(smem_u32(&bar), 0u, &abort_flag, limit_ns);
    if (gave_up) *gave_up = ok ? 0u : 1u;
  }
}

// ----------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// 2-D uint8 tensor [outer, inner] (inner contiguous, row pitch ld bytes), boxes of
// {128 bytes, box_outer rows}, 128-byte swizzle, out-of-bounds reads return zero.
bool make_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld, int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld};
  cuuint32_t box[2] = {128u, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 2-D output tensor [rows, cols] of bf16 or fp32, boxes of {128 bytes, 32 rows}, 128-byte swizzle.
// Packed 4-bit elements, two per byte, [outer rows] x [inner elements], row pitch ld_bytes: the load expands every 16
// elements (8 bytes) to a 16-byte group in shared memory, so a box of 128 elements fills the same 128-byte swizzled
// row as 128 one-byte elements and the kernels' stage layout and descriptors stay as they are.
bool make_map_packed4(CUtensorMap* map, const void* base, int64_t inner_elems, int64_t outer, int64_t ld_bytes,
                      int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner_elems, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld_bytes};
  cuuint32_t box[2] = {128u, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_out_map(CUtensorMap* map, void* base, int64_t cols, int64_t rows, int64_t ld, bool f32) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t esz = f32 ? 4 : 2;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
  cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 2-D FP8 output [rows, cols] (one byte per element): boxes of {64 bytes, 32 rows}, 64-byte swizzle.
bool make_q_map(CUtensorMap* map, void* base, int64_t cols, int64_t rows, int64_t ld) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld};
  cuuint32_t box[2] = {64u, 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Operand format beyond the public FP8 enum: 4-bit E2M1 elements, which kind::f8f6f4 reads from shared memory in
// 16-byte groups of 16 elements (8 bytes of codes, 8 of padding) -- the form a tensor map of the packed 4-bit type
// expands them to on the way in.
constexpr int kFmtE2M1 = 2;

uint32_t make_idesc(int fmt_a, int fmt_b, bool a_mn, bool b_mn, int n, int m = BM) {
  // [4,6) accumulator format (1 = fp32)   [7,10) A format   [10,13) B format (0 = E4M3, 1 = E5M2, 5 = E2M1)
  // [15] A major (1 = MN)   [16] B major   [17,23) N >> 3   [24,29) M >> 4
  auto code = [](int f) { return f == TWEO_E5M2 ? 1u : (f == kFmtE2M1 ? 5u : 0u); };
  uint32_t d = 0;
  d |= 1u << 4;
  d |= code(fmt_a) << 7;
  d |= code(fmt_b) << 10;
  d |= (uint32_t)(a_mn ? 1 : 0) << 15;
  d |= (uint32_t)(b_mn ? 1 : 0) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(m >> 4) << 24;
  return d;
}

// Band height of the tile numbering: the `workers` tiles in flight cover about g x workers/g
// tiles, so g near sqrt(workers) keeps the rows of A and the columns of B they touch smallest.
int raster_band(int tiles_m, int workers) {
  int g = 1;
  while ((g + 1) * (g + 1) <= workers) ++g;
  if (g > tiles_m) g = tiles_m;
  return g < 1 ? 1 : g;
}

template <int BN, bool A_MN, bool B_MN, int STAGES, bool OUT_F32>
tweo_status_t launch_cfg(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, GemmParams& p,
                         void* ws, size_t ws_bytes, cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * (BM * BK + BN * BK) + 4 * 2 * 32 * 128 + 1024 + 256;
  auto kern = gemm_fp8_kernel<BN, A_MN, B_MN, STAGES, OUT_F32>;
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    device_once_done(attr_done, attr_dev);
  }
  p.tiles_m = (p.Md + BM - 1) / BM;
  p.tiles_n = (p.Nd + BN - 1) / BN;
  p.k_blocks = (p.Kc + BK - 1) / BK;
  const int tiles = p.tiles_m * p.tiles_n;
  const int sms = sm_count();
  int grid = sms < tiles ? sms : tiles;
  p.raster_g = raster_band(p.tiles_m, sms);
  p.sk_tiles = 0;
  p.sk_partials = nullptr;
  p.sk_counters = nullptr;
  // Stream-K when whole-tile dealing would idle more than ~15 % of the SM-time and the
  // contraction is long enough to pay for the fix-up (a 128 x BN fp32 round trip through L2).
  const size_t sk_need = kWsPartialsOffset + (size_t)sms * kWsPartialBytesPerSm;
  const int waves = (tiles + sms - 1) / sms;
  if (ws && ws_bytes >= sk_need && aligned16(ws) && p.k_blocks >= 12 &&
      (double)tiles < 0.85 * (double)waves * sms) {
    const int full = tiles / sms;
    p.sk_tiles = full == 0 ? tiles : tiles - (full - 1) * sms;
    if ((size_t)p.sk_tiles * 4 * sizeof(uint32_t) > kWsPartialsOffset - kWsCountersOffset) p.sk_tiles = 0;  // counters
  }
  if (p.sk_tiles > 0) {
    grid = sms;
    if ((int64_t)p.sk_tiles * p.k_blocks < grid) grid = (int)((int64_t)p.sk_tiles * p.k_blocks);
    p.sk_counters = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(ws) + kWsCountersOffset);
    p.sk_partials = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + kWsPartialsOffset);
  }
  kern<<<grid, kThreads, smem, st>>>(ma, mb, md, p);
  count_launch();
  return check_launch("gemm_fp8_kernel");
}

// How many of the `tiles` the pair kernel splits along the contraction (0 = none).  Whole tiles
// are dealt round-robin; what does not fill the last wave is split so that every pair gets the
// same number of k-blocks.  Parking and re-adding 256 x 256 fp32 accumulators costs each SM
// tens of microseconds' worth of L2 traffic spread over the GPU (measured: about 25 000 cycles
// per pair), so the split only pays when the idle time it removes is clearly larger.
int pair_split_tiles(int tiles, int workers, int k_blocks) {
  const int rem = tiles % workers;
  if (rem == 0) return 0;
  const double idle_clks = (double)(workers - rem) / workers * k_blocks * 512.0;  // per pair, if not split
  if (idle_clks < 40000.0) return 0;
  if ((int64_t)rem * k_blocks < (int64_t)8 * workers) return 0;                  // shares of at least 8 k-blocks
  return rem;
}

template <bool A_MN, bool B_MN, bool OUT_F32>
tweo_status_t launch_pair(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, GemmParams& p,
                          void* ws, size_t ws_bytes, cudaStream_t st) {
  constexpr int STAGES = 6;
  constexpr size_t smem = (size_t)STAGES * (BM * BK + 128 * BK) + 4 * 2 * 32 * 128 + 1024 + 256;
  if (p.out_amax || p.out_q) return TWEO_ERR_INVALID_ARG;  // fused outputs belong to the staged instantiations
  auto kern = gemm_fp8_pair_kernel<A_MN, B_MN, STAGES, OUT_F32>;
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 0));
    device_once_done(attr_done, attr_dev);
  }
  p.tiles_m = (p.Md + 2 * BM - 1) / (2 * BM);
  p.tiles_n = (p.Nd + 255) / 256;
  p.k_blocks = (p.Kc + BK - 1) / BK;
  p.sk_tiles = 0;
  p.sk_partials = nullptr;
  p.sk_counters = nullptr;
  const int tiles = p.tiles_m * p.tiles_n;
  const int sms = sm_count();
  int pairs = sms / 2;
  p.raster_g = raster_band(p.tiles_m, pairs);
  if (ws && ws_bytes >= kWsPartialsOffset + (size_t)sms * kWsPartialBytesPerSm && aligned16(ws)) {
    p.sk_tiles = pair_split_tiles(tiles, pairs, p.k_blocks);
    if (p.sk_tiles > 0) {
      p.sk_counters = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(ws) + kWsCountersOffset);
      p.sk_partials = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + kWsPartialsOffset);
    }
  }
  if (p.sk_tiles == 0 && pairs > tiles) pairs = tiles;
  TWEO_CUDA_TRY(launch_chain(kern, dim3((unsigned)(2 * pairs)), dim3(kThreads), smem, st, 2, ma, mb, md, md, p));
  count_launch();
  return check_launch("gemm_fp8_pair_kernel");
}

struct Operand {
  const uint8_t* ptr;
  int64_t ld;
  int fmt;
  bool mn_major;  // stored [Kc, rows] (true) or [rows, Kc] (false)
};

// D[Md,Nd] = A . B, see the header comment for how the three linear products map here.
tweo_status_t run_gemm(const Operand& A, const Operand& B, int64_t Md, int64_t Nd, int64_t Kc, GemmParams p,
                       void* ws, size_t ws_bytes, cudaStream_t st) {
  if (Md < 1 || Nd < 1 || Kc < 1) return TWEO_ERR_INVALID_ARG;
  if (Md > INT32_MAX || Nd > INT32_MAX || Kc > INT32_MAX) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(A.ptr) || !aligned16(B.ptr) || !aligned16(p.d) || (A.ld & 15) || (B.ld & 15))
    return TWEO_ERR_ALIGNMENT;
  if ((p.ldd * (p.out_f32 ? 4 : 2)) & 15) return TWEO_ERR_ALIGNMENT;
  p.Md = (int32_t)Md;
  p.Nd = (int32_t)Nd;
  p.Kc = (int32_t)Kc;
  const int BN = Nd > 128 ? 256 : 128;
  // CTA pairs (256 x 256 tiles) whenever the output has more than one 128-row block and is wide enough
  const bool use_pair = Md > 128 && Nd > 128;
  p.idesc = use_pair ? make_idesc(A.fmt, B.fmt, A.mn_major, B.mn_major, 256, 256)
                     : make_idesc(A.fmt, B.fmt, A.mn_major, B.mn_major, BN);

  CUtensorMap ma, mb, md;
  bool ok = make_out_map(&md, p.d, Nd, Md, p.ldd, p.out_f32 != 0);
  if (!ok) {
    cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled (output)");
    return TWEO_ERR_CUDA;
  }
  if (A.mn_major) ok = make_map(&ma, A.ptr, Md, Kc, A.ld, BK);   // [Kc, Md]: box 128 (Md) x BK rows
  else ok = make_map(&ma, A.ptr, Kc, Md, A.ld, BM);              // [Md, Kc]: box 128 (Kc) x BM rows
  if (B.mn_major) ok = ok && make_map(&mb, B.ptr, Nd, Kc, B.ld, BK);
  else ok = ok && make_map(&mb, B.ptr, Kc, Nd, B.ld, use_pair ? 128 : BN);  // a pair CTA loads half of B
  if (!ok) {
    cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return TWEO_ERR_CUDA;
  }
  if (p.out_amax) {
    TWEO_CUDA_TRY(launch_chain(zero_float_kernel, dim3(1), dim3(1), 0, st, 0, p.out_amax));
    count_launch();
  }
  if (use_pair) {
#define TWEO_PAIR(AMN, BMN) (p.out_f32 ? launch_pair<AMN, BMN, true>(ma, mb, md, p, ws, ws_bytes, st) : launch_pair<AMN, BMN, false>(ma, mb, md, p, ws, ws_bytes, st))
    if (!A.mn_major && !B.mn_major) return TWEO_PAIR(false, false);
    if (!A.mn_major && B.mn_major) return TWEO_PAIR(false, true);
    if (A.mn_major && B.mn_major) return TWEO_PAIR(true, true);
    return TWEO_ERR_INVALID_ARG;
#undef TWEO_PAIR
  }
#define TWEO_DISPATCH(AMN, BMN)                                                                   \
  (p.out_f32 ? (BN == 256 ? launch_cfg<256, AMN, BMN, 4, true>(ma, mb, md, p, ws, ws_bytes, st)                 \
                          : launch_cfg<128, AMN, BMN, 6, true>(ma, mb, md, p, ws, ws_bytes, st))                \
             : (BN == 256 ? launch_cfg<256, AMN, BMN, 4, false>(ma, mb, md, p, ws, ws_bytes, st)                \
                          : launch_cfg<128, AMN, BMN, 6, false>(ma, mb, md, p, ws, ws_bytes, st)))
  if (!A.mn_major && !B.mn_major) return TWEO_DISPATCH(false, false);
  if (!A.mn_major && B.mn_major) return TWEO_DISPATCH(false, true);
  if (A.mn_major && B.mn_major) return TWEO_DISPATCH(true, true);
  return TWEO_ERR_INVALID_ARG;
#undef TWEO_DISPATCH
}

// Forward product (or data gradient) with the MLP activation and / or the FP8 copy of the output in the
// epilogue (pair kernel only; every tile whole; the FP8 copy staged through shared memory).
// EPIW epilogue warps, STAGES operand stages, EBUF staging buffers per epilogue warp.
template <int ACT, bool B_MN, int EPIW, int STAGES, int EBUF>
tweo_status_t launch_pair_act_cfg(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md,
                                  const CUtensorMap& mq, GemmParams& p, cudaStream_t st) {
  constexpr int THREADS = 64 + 32 * EPIW;
  constexpr size_t smem =
      (size_t)STAGES * (BM * BK + 128 * BK) + EPIW * EBUF * 32 * 128 + EPIW * EBUF * 32 * 64 + 1024 + 256;
  static_assert(smem <= 227 * 1024, "shared memory per CTA");
  auto kern = gemm_fp8_pair_kernel<false, B_MN, STAGES, false, false, ACT, true, EPIW, EBUF>;
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    device_once_done(attr_done, attr_dev);
  }
  p.tiles_m = (p.Md + 2 * BM - 1) / (2 * BM);
  p.tiles_n = ACT == 3 ? (p.Nd + 127) / 128 : (p.Nd + 255) / 256;
  p.k_blocks = (p.Kc + BK - 1) / BK;
  p.sk_tiles = 0;
  p.sk_partials = nullptr;
  p.sk_counters = nullptr;
  const int tiles = p.tiles_m * p.tiles_n;
  int pairs = sm_count() / 2;
  p.raster_g = raster_band(p.tiles_m, pairs);
  if (pairs > tiles) pairs = tiles;
  TWEO_CUDA_TRY(launch_chain(kern, dim3((unsigned)(2 * pairs)), dim3(THREADS), smem, st, 2, ma, mb, md, mq, p));
  count_launch();
  return check_launch("gemm_fp8_pair_kernel (fused epilogue)");
}

// Which configuration a product with a per-element epilogue takes (measured on B200, microseconds, forward
// product with bf16 + amax + FP8 outputs; (epilogue warps, operand stages, staging buffers)):
//   [8192x768].[2304x768]^T    (8,4,2) 19.3  (4,5,2) 19.1  (8,5,1) 18.3  (4,6,1) 20.7
//   [16384x2048].[6144x2048]^T (8,4,2) 169.6 (4,5,2) 158.7 (8,5,1) 161.9 (4,6,1) 156.9
// Short contractions are bound by the epilogue's issue rate (eight warps), long ones by the main loop, which
// wants the deepest operand ring; one staging buffer per warp pays for the extra stage in both.
template <int ACT, bool B_MN = false>
tweo_status_t launch_pair_act(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md,
                              const CUtensorMap& mq, GemmParams& p, cudaStream_t st) {
  if (ACT == 3 || (p.Kc + BK - 1) / BK >= 16)          // SwiGLU (238 registers) always takes four warps
    return launch_pair_act_cfg<ACT, B_MN, 4, 6, 1>(ma, mb, md, mq, p, st);
  return launch_pair_act_cfg<(ACT == 3 ? 0 : ACT), B_MN, 8, 5, 1>(ma, mb, md, mq, p, st);
}

// D[M,N] = A[M,K] . B with A stored [M,K]; B stored [N,K] (w_mn false: the forward product) or [K,N] (w_mn
// true: the data gradient, which reads the weight in its forward layout; plain epilogue only).
// N: output columns, K: contraction.  SwiGLU: wq has 2 N rows (gate rows, then up rows).
tweo_status_t run_fwd_act(const uint8_t* xq, int64_t ldx, int fmt_x, const uint8_t* wq, int64_t ldw, int fmt_w,
                          bool w_mn, int act, int64_t M, int64_t N, int64_t K, GemmParams p, cudaStream_t st) {
  if (w_mn && act != TWEO_ACT_NONE) return TWEO_ERR_INVALID_ARG;
  if (M > INT32_MAX || 2 * N > INT32_MAX || K > INT32_MAX) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(xq) || !aligned16(wq) || !aligned16(p.d) || (ldx & 15) || (ldw & 15) || ((p.ldd * 2) & 15))
    return TWEO_ERR_ALIGNMENT;
  p.Md = (int32_t)M;
  p.Nd = (int32_t)N;
  p.Kc = (int32_t)K;
  p.idesc = make_idesc(fmt_x, fmt_w, false, w_mn, 256, 256);
  CUtensorMap ma, mb, md, mq;
  // without a bf16 output the store is skipped; the map then describes the FP8 output's memory and is never used
  bool ok = p.d ? make_out_map(&md, p.d, N, M, p.ldd, false) : make_out_map(&md, p.out_q, N / 2, M, p.ldq / 2, false);
  if (p.out_q) ok = ok && make_q_map(&mq, p.out_q, N, M, p.ldq);
  else mq = md;
  ok = ok && make_map(&ma, xq, K, M, ldx, BM);
  if (w_mn) ok = ok && make_map(&mb, wq, N, K, ldw, BK);
  else ok = ok && make_map(&mb, wq, K, act == TWEO_ACT_SWIGLU ? 2 * N : N, ldw, 128);
  if (!ok) {
    cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return TWEO_ERR_CUDA;
  }
  if (p.out_amax) {
    TWEO_CUDA_TRY(launch_chain(zero_float_kernel, dim3(1), dim3(1), 0, st, 0, p.out_amax));
    count_launch();
  }
  switch (act) {
    case TWEO_ACT_NONE:
      return w_mn ? launch_pair_act<0, true>(ma, mb, md, mq, p, st) : launch_pair_act<0>(ma, mb, md, mq, p, st);
    case TWEO_ACT_GELU: return launch_pair_act<1>(ma, mb, md, mq, p, st);
    case TWEO_ACT_GELU_TANH: return launch_pair_act<2>(ma, mb, md, mq, p, st);
    case TWEO_ACT_SWIGLU: return launch_pair_act<3>(ma, mb, md, mq, p, st);
    default: return TWEO_ERR_INVALID_ARG;
  }
}

// Forward product for M <= 128 (see gemm_skinny.cuh): W is streamed once, K is sliced over CTAs.  The caller has
// filled the scale fields of `p`; this fills the shape, the ring and the slicing, and launches.
// w_packed4: W holds packed E2M1 codes (two per byte, ldw in BYTES); the ring and the kernel are the same, only the
// tensor map of W differs (and the operand format in p.idesc, set by the caller).
template <bool I8>
tweo_status_t launch_skinny(SkinnyParams& p, const void* xq, int64_t ldx, const void* wq, int64_t ldw, int64_t M, int64_t N,
                            int64_t K, cudaStream_t st, bool w_packed4 = false) {
  if (N > INT32_MAX || K > INT32_MAX) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(xq) || !aligned16(wq) || (ldx & 15) || (ldw & 15)) return TWEO_ERR_ALIGNMENT;
  if (w_packed4 && ((reinterpret_cast<uintptr_t>(wq) & 31u) || (ldw & 31) || (K & 127))) return TWEO_ERR_ALIGNMENT;
  p.M = (int32_t)M;
  p.N = (int32_t)N;
  p.Mpad = (int32_t)((M + 15) / 16 * 16);
  p.k_blocks = (int32_t)((K + BK - 1) / BK);
  p.stage_bytes = (uint32_t)((BM * BK + p.Mpad * 128 + 1023) / 1024 * 1024);
  p.w_tx_bytes = (uint32_t)(w_packed4 ? BM * BK / 2 : BM * BK);
  // A ring of at most 100 KB, so that two CTAs fit an SM: the CTAs of the next kernel of a launch chain become
  // resident (and fetch their first ring of W) while this kernel's are still reducing and writing.
  p.stages = (int32_t)((100 * 1024) / p.stage_bytes);
  if (p.stages > kSkinnyMaxStages) p.stages = kSkinnyMaxStages;
  if (p.stages < 2) p.stages = 2;
  p.tmem_cols = p.Mpad <= 32 ? 32u : (p.Mpad <= 64 ? 64u : 128u);
  const int sms = sm_count();
  const int slabs = (int)((N + 127) / 128);
  // slices of K per slab = CTAs per cluster: the largest count up to the portable cluster size that keeps the grid
  // within two CTAs per SM and leaves every slice at least four k-blocks
  p.slices = 1;
  for (int sl = 2; sl <= 8; ++sl)
    if (slabs * sl <= 2 * sms && p.k_blocks / sl >= 4) p.slices = sl;
  CUtensorMap mw, mx;
  const bool w_ok = w_packed4 ? make_map_packed4(&mw, wq, K, N, ldw, BM) : make_map(&mw, wq, K, N, ldw, BM);
  if (!w_ok || !make_map(&mx, xq, K, M, ldx, p.Mpad)) {
    cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return TWEO_ERR_CUDA;
  }
  const size_t smem = (size_t)p.stages * p.stage_bytes + 1024 + 256;
  auto kern = gemm_fp8_skinny_kernel<I8>;
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(100 * 1024 + 1024 + 256)));
    device_once_done(attr_done, attr_dev);
  }
  TWEO_CUDA_TRY(launch_chain(kern, dim3((unsigned)(slabs * p.slices)), dim3(kThreads), smem, st, (unsigned)p.slices, mw,
                             mx, p));
  count_launch();
  return check_launch("gemm_fp8_skinny_kernel");
}

tweo_status_t run_skinny(const uint8_t* xq, int64_t ldx, int fmt_x, const uint8_t* wq, int64_t ldw, int fmt_w,
                         const float* sx_inv, const float* sw_inv, bool sx_is_scale, uint16_t* y, int64_t ldy, int64_t M,
                         int64_t N, int64_t K, cudaStream_t st) {
  SkinnyParams p{};
  p.y = y;
  p.ldy = ldy;
  p.idesc = make_idesc(fmt_w, fmt_x, false, false, (int)((M + 15) / 16 * 16), BM);
  p.sx_inv = sx_inv;
  p.sw_inv = sw_inv;
  p.sx_is_scale = sx_is_scale ? 1 : 0;
  return launch_skinny<false>(p, xq, ldx, wq, ldw, M, N, K, st);
}

// The same with W as packed E2M1 codes: half the bytes of the stream that bounds the call.
tweo_status_t run_skinny_w4(const uint8_t* xq, int64_t ldx, int fmt_x, const uint8_t* w4, int64_t ldw_bytes,
                            const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M, int64_t N,
                            int64_t K, cudaStream_t st) {
  SkinnyParams p{};
  p.y = y;
  p.ldy = ldy;
  p.idesc = make_idesc(kFmtE2M1, fmt_x, false, false, (int)((M + 15) / 16 * 16), BM);
  p.sx_inv = sx_inv;
  p.sw_inv = sw_inv;
  p.sx_is_scale = 0;
  return launch_skinny<false>(p, xq, ldx, w4, ldw_bytes, M, N, K, st, true);
}

// Up to kGroupMaxProblems independent products in ONE launch of the CTA-pair kernel (see gemm_pair_group.cuh).
// D[Md,Nd] = A . B over Kc; A stored [Md,Kc] (a_mn false) or [Kc,Md]; B stored [Nd,Kc] (b_mn false) or [Kc,Nd].
struct GroupDesc {
  const uint8_t *a, *b;
  int64_t lda, ldb, Md, Nd, Kc;
  int fa, fb;
  bool a_mn, b_mn;
  uint16_t* d;
  int64_t ldd;
  const float *sa, *sb;
  // fused epilogue (all optional): amax of the bf16 output, its FP8 copy with the scale *q_scale
  float* out_amax = nullptr;
  uint8_t* out_q = nullptr;
  int64_t ldq = 0;
  int q_fmt = TWEO_E4M3;
  const float* q_scale = nullptr;
};

struct FloatPtrs {
  float* p[kGroupMaxProblems];
  int n;
};
// Clears the amax cells of a group's fused epilogues (in the chain, like zero_float_kernel).
__global__ void zero_floats_kernel(const FloatPtrs f) {
  chain_release();
  chain_wait();
  if ((int)threadIdx.x < f.n) *f.p[threadIdx.x] = 0.0f;
}

// QST: fused epilogue outputs (amax, FP8 copy) on some products.  EPIW / EBUF as in the kernel; the operand ring
// takes what the staging buffers leave of the shared memory.
template <int LIST, bool QST, int EPIW, int EBUF>
tweo_status_t run_group_list(GroupDesc* d, int n, cudaStream_t st) {
  constexpr size_t staging = (size_t)EPIW * EBUF * (32 * 128 + (QST ? 32 * 64 : 0));
  constexpr int STAGES = (int)((227 * 1024 - 1024 - 256 - staging) / (BM * BK + 128 * BK)) > 6
                             ? 6 : (int)((227 * 1024 - 1024 - 256 - staging) / (BM * BK + 128 * BK));
  static_assert(STAGES >= 4, "operand ring too short");
  constexpr size_t smem = (size_t)STAGES * (BM * BK + 128 * BK) + staging + 1024 + 256;
  auto kern = gemm_fp8_pair_group_kernel<STAGES, LIST, QST, EPIW, EBUF>;
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    device_once_done(attr_done, attr_dev);
  }
  const int pairs_all = sm_count() / 2;
  static thread_local PairGroupParams<LIST> g;   // 8 - 20 KB: kept off the stack
  g.n_problems = n;
  int cost[kGroupMaxProblems];
  g.tile_start[0] = 0;
  for (int i = 0; i < n; ++i) {
    GroupProblem& q = g.pr[i];
    q.Md = (int32_t)d[i].Md;
    q.Nd = (int32_t)d[i].Nd;
    q.tiles_m = (int32_t)((d[i].Md + 2 * BM - 1) / (2 * BM));
    q.tiles_n = (int32_t)((d[i].Nd + 255) / 256);
    q.k_blocks = (int32_t)((d[i].Kc + BK - 1) / BK);
    q.raster_g = raster_band(q.tiles_m, pairs_all);
    q.a_mn = d[i].a_mn ? 1 : 0;
    q.b_mn = d[i].b_mn ? 1 : 0;
    q.idesc = make_idesc(d[i].fa, d[i].fb, d[i].a_mn, d[i].b_mn, 256, 256);
    q.sa_inv = d[i].sa;
    q.sb_inv = d[i].sb;
    q.out_amax = d[i].out_amax;
    q.q_scale = d[i].out_q ? d[i].q_scale : nullptr;
    q.q_fmt = d[i].q_fmt;
    q.pad = 0;
    g.tile_start[i + 1] = g.tile_start[i] + q.tiles_m * q.tiles_n;
    cost[i] = (q.k_blocks < 8 ? 8 : q.k_blocks) + 2;  // k-blocks, with a floor for the epilogue of short tiles
    bool ok = make_out_map(&g.md[i], d[i].d, d[i].Nd, d[i].Md, d[i].ldd, false);
    if (QST && d[i].out_q) ok = ok && make_q_map(&g.mq[i], d[i].out_q, d[i].Nd, d[i].Md, d[i].ldq);
    else g.mq[i] = g.md[i];
    if (d[i].a_mn) ok = ok && make_map(&g.ma[i], d[i].a, d[i].Md, d[i].Kc, d[i].lda, BK);
    else ok = ok && make_map(&g.ma[i], d[i].a, d[i].Kc, d[i].Md, d[i].lda, BM);
    if (d[i].b_mn) ok = ok && make_map(&g.mb[i], d[i].b, d[i].Nd, d[i].Kc, d[i].ldb, BK);
    else ok = ok && make_map(&g.mb[i], d[i].b, d[i].Kc, d[i].Nd, d[i].ldb, 128);   // a pair CTA loads half of B
    if (!ok) {
      cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
      return TWEO_ERR_CUDA;
    }
  }
  for (int i = n; i <= kGroupMaxProblems; ++i) g.tile_start[i] = g.tile_start[n];
  g.total_tiles = g.tile_start[n];
  g.pad = 0;
  int pairs = pairs_all < g.total_tiles ? pairs_all : g.total_tiles;
  g.use_lists = (g.total_tiles <= LIST && pairs <= kGroupMaxPairs) ? 1 : 0;
  if (g.use_lists) {
    // longest processing time first: every tile goes to the pair with the least work so far
    typedef std::pair<int64_t, int> Load;  // (work, pair); smallest on top, ties to the lower pair index
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int p = 0; p < pairs; ++p) heap.push(Load(0, p));
    static thread_local uint8_t owner[LIST];
    int count[kGroupMaxPairs + 1] = {0};
    int prob = 0;
    for (int t = 0; t < g.total_tiles; ++t) {
      while (t >= g.tile_start[prob + 1]) ++prob;
      Load l = heap.top();
      heap.pop();
      owner[t] = (uint8_t)l.second;
      ++count[l.second];
      l.first += cost[prob];
      heap.push(l);
    }
    int fill[kGroupMaxPairs + 1];
    g.first[0] = 0;
    for (int p = 0; p < pairs; ++p) {
      g.first[p + 1] = (uint16_t)(g.first[p] + count[p]);
      fill[p] = g.first[p];
    }
    for (int t = 0; t < g.total_tiles; ++t) g.list[fill[owner[t]]++] = (uint16_t)t;  // ascending t within a pair
  }
  if (QST) {
    FloatPtrs z;
    z.n = 0;
    for (int i = 0; i < n; ++i)
      if (d[i].out_amax) z.p[z.n++] = d[i].out_amax;
    if (z.n) {
      TWEO_CUDA_TRY(launch_chain(zero_floats_kernel, dim3(1), dim3(32), 0, st, 0, z));
      count_launch();
    }
  }
  TWEO_CUDA_TRY(launch_chain(kern, dim3((unsigned)(2 * pairs)), dim3(64 + 32 * EPIW), smem, st, 2, g));
  count_launch();
  return check_launch("gemm_fp8_pair_group_kernel");
}

tweo_status_t run_group(GroupDesc* d, int n, cudaStream_t st) {
  if (n < 1 || n > kGroupMaxProblems) return TWEO_ERR_INVALID_ARG;
  // the products with the longer tiles go first in the tile list (stable: equal lengths keep the caller's order)
  std::stable_sort(d, d + n, [](const GroupDesc& x, const GroupDesc& y) {
    return (x.Kc + BK - 1) / BK > (y.Kc + BK - 1) / BK;
  });
  int64_t tiles = 0;
  for (int i = 0; i < n; ++i) tiles += ((d[i].Md + 2 * BM - 1) / (2 * BM)) * ((d[i].Nd + 255) / 256);
  bool fused = false;
  int64_t fused_kb_min = INT64_MAX;
  for (int i = 0; i < n; ++i)
    if (d[i].out_amax || d[i].out_q) {
      fused = true;
      fused_kb_min = std::min(fused_kb_min, (d[i].Kc + BK - 1) / BK);
    }
  const bool small = tiles <= kGroupListSmall;
  if (!fused)
    return small ? run_group_list<kGroupListSmall, false, 4, 2>(d, n, st) : run_group_list<kGroupListLarge, false, 4, 2>(d, n, st);
  // the fused epilogue computes per element: at short contractions it outlasts the tile's main loop unless eight
  // warps share it (the rule of the single fused products)
  if (fused_kb_min < 16)
    return small ? run_group_list<kGroupListSmall, true, 8, 1>(d, n, st) : run_group_list<kGroupListLarge, true, 8, 1>(d, n, st);
  return small ? run_group_list<kGroupListSmall, true, 4, 1>(d, n, st) : run_group_list<kGroupListLarge, true, 4, 1>(d, n, st);
}

// dX and dW of one linear layer as a group of two products.
tweo_status_t run_bwd_group(const uint8_t* dyq, int64_t lddy, int fmt_dy, const uint8_t* xq, int64_t ldx, int fmt_x,
                            const uint8_t* wq, int64_t ldw, int fmt_w, const float* sdy_inv, const float* sx_inv,
                            const float* sw_inv, uint16_t* dx, int64_t lddx, uint16_t* dw, int64_t lddw, int64_t M,
                            int64_t N, int64_t K, cudaStream_t st) {
  // product D: dX[M,K] = dYq[M,N] . Wq[N,K] (contraction N); product W: dW[N,K] = dYq^T . Xq (contraction M)
  GroupDesc d[2] = {{dyq, wq, lddy, ldw, M, K, N, fmt_dy, fmt_w, false, true, dx, lddx, sdy_inv, sw_inv},
                    {dyq, xq, lddy, ldx, N, K, M, fmt_dy, fmt_x, true, true, dw, lddw, sdy_inv, sx_inv}};
  return run_group(d, 2, st);
}

bool fmt_ok(int f) { return f == TWEO_E4M3 || f == TWEO_E5M2; }

tweo_status_t fill_epilogue(GemmParams& p, const tweo_epilogue_t* epi) {
  p.out_amax = nullptr;
  p.out_q = nullptr;
  p.ldq = 0;
  p.q_fmt = TWEO_E4M3;
  p.q_scale = nullptr;
  if (!epi) return TWEO_OK;
  p.out_amax = epi->out_amax;
  if (epi->out_q) {
    if (!epi->q_scale || !fmt_ok(epi->q_fmt)) return TWEO_ERR_INVALID_ARG;
    if (!aligned16(epi->out_q) || (epi->ldq & 15)) return TWEO_ERR_ALIGNMENT;
    p.out_q = epi->out_q;
    p.ldq = epi->ldq;
    p.q_fmt = epi->q_fmt;
    p.q_scale = epi->q_scale;
  }
  return TWEO_OK;
}

}  // namespace

namespace tweo_detail {

tweo_status_t read_and_clear_device_status(cudaStream_t stream) {
  TWEO_CUDA_TRY(cudaStreamSynchronize(stream));
  unsigned int v = 0, zero = 0;
  TWEO_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_device_status, sizeof v));
  if (v != 0) TWEO_CUDA_TRY(cudaMemcpyToSymbol(g_device_status, &zero, sizeof zero));
  return v == 0 ? TWEO_OK : (tweo_status_t)v;
}

// Device address of the status word on the current device, for kernels in other files whose
// bounded waits report through it (nullptr if the lookup fails).
unsigned int* device_status_word() {
  static unsigned int* cached[64] = {nullptr};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_device_status) != cudaSuccess) return nullptr;
    cached[dev] = static_cast<unsigned int*>(ptr);
  }
  return cached[dev];
}

// Used by the static W8A8 entry point: forward product on already-cast activations.
tweo_status_t gemm_fwd_codes(const uint8_t* xq, int64_t ldx, int fmt_x, const uint8_t* wq, int64_t ldw, int fmt_w,
                             const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                             int64_t N, int64_t K, const tweo_epilogue_t* epi, void* ws, size_t ws_bytes,
                             cudaStream_t st, bool sx_is_scale) {
  const bool fused = epi && (epi->out_amax || epi->out_q);
  if (M <= 128 && !fused)  // few tokens: stream W once, tokens on the MMA's N side
    return run_skinny(xq, ldx, fmt_x, wq, ldw, fmt_w, sx_inv, sw_inv, sx_is_scale, y, ldy, M, N, K, st);
  GemmParams p{};
  p.d = y;
  p.ldd = ldy;
  p.sa_inv = sx_inv;
  p.sb_inv = sw_inv;
  p.sa_is_scale = sx_is_scale ? 1 : 0;
  tweo_status_t s = fill_epilogue(p, epi);
  if (s != TWEO_OK) return s;
  if (fused && M > 128 && N > 128)  // extra outputs leave through shared memory and TMA
    return run_fwd_act(xq, ldx, fmt_x, wq, ldw, fmt_w, false, TWEO_ACT_NONE, M, N, K, p, st);
  return run_gemm(Operand{xq, ldx, fmt_x, false}, Operand{wq, ldw, fmt_w, false}, M, N, K, p, ws, ws_bytes, st);
}

// The integer (Eq. 4) linear on the pair kernel: bf16 output (y), or 8-bit output requantised with the
// static scale *sy (yq) -- exactly one of the two.
tweo_status_t run_int8_linear(const int8_t* xq, int64_t ldx, const float* sx, int32_t sx_per_row, const int8_t* wq,
                              int64_t ldw, const float* sw, int32_t sw_per_row, int32_t bits, uint16_t* y, int64_t ldy,
                              int8_t* yq, int64_t ldq, const float* sy, int64_t M, int64_t N, int64_t K,
                              cudaStream_t stream) {
  if (!xq || !wq || !sx || !sw || bits < 2 || bits > 8) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(xq) || !aligned16(wq) || (ldx & 15) || (ldw & 15)) return TWEO_ERR_ALIGNMENT;
  if (y && (!aligned16(y) || (ldy & 7))) return TWEO_ERR_ALIGNMENT;
  if (yq && (!aligned16(yq) || (ldq & 15))) return TWEO_ERR_ALIGNMENT;
  const bool q8 = yq != nullptr;
  if (!q8 && M <= 128) {
    // few tokens (small-batch inference, Sec. 4.4): the weight-streaming kernel with integer operands
    const int Q_ = (1 << (bits - 1)) - 1;
    const int Mpad = (int)((M + 15) / 16 * 16);
    SkinnyParams sp{};
    sp.y = y;
    sp.ldy = ldy;
    // kind::i8 descriptor: int32 accumulators, signed 8-bit A and B, K-major, M = 128 (rows of W), N = padded tokens
    sp.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(Mpad >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    sp.row_scale = sx;
    sp.col_scale = sw;
    sp.row_scale_per_row = sx_per_row ? 1 : 0;
    sp.col_scale_per_col = sw_per_row ? 1 : 0;
    sp.post_scale = 1.0f / ((float)Q_ * (float)Q_);
    return launch_skinny<true>(sp, xq, ldx, wq, ldw, M, N, K, stream);
  }
  constexpr size_t smem6 = (size_t)6 * (BM * BK + 128 * BK) + 4 * 2 * 32 * 128 + 1024 + 256;
  constexpr size_t smem5q = (size_t)5 * (BM * BK + 128 * BK) + 4 * 2 * 32 * 128 + 4 * 2 * 32 * 64 + 1024 + 256;
  auto kern_bf16 = gemm_fp8_pair_kernel<false, false, 6, false, true>;
  auto kern_q8 = gemm_fp8_pair_kernel<false, false, 5, false, true, 0, true>;
  static std::atomic<uint64_t> attr_done{0};  // per device
  int attr_dev = 0;
  if (device_once_pending(attr_done, &attr_dev)) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem6));
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern_q8, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem5q));
    device_once_done(attr_done, attr_dev);
  }
  GemmParams p{};
  p.d = y;
  p.ldd = ldy;
  p.Md = (int32_t)M;
  p.Nd = (int32_t)N;
  p.Kc = (int32_t)K;
  p.tiles_m = (int32_t)((M + 2 * BM - 1) / (2 * BM));
  p.tiles_n = (int32_t)((N + 255) / 256);
  p.k_blocks = (int32_t)((K + BK - 1) / BK);
  const int tiles = p.tiles_m * p.tiles_n;
  int pairs = sm_count() / 2;
  p.raster_g = raster_band(p.tiles_m, pairs);
  if (pairs > tiles) pairs = tiles;
  const float Q = (float)((1 << (bits - 1)) - 1);
  p.row_scale = sx;
  p.col_scale = sw;
  p.row_scale_per_row = sx_per_row ? 1 : 0;
  p.col_scale_per_col = sw_per_row ? 1 : 0;
  p.post_scale = 1.0f / (Q * Q);
  p.q8_qmax = Q;
  if (q8) {
    p.out_q = reinterpret_cast<uint8_t*>(yq);
    p.ldq = ldq;
    p.q_scale = sy;
  }
  // instruction descriptor of kind::i8: int32 accumulators, signed 8-bit A and B, K-major, N = 256, M = 256
  p.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
  CUtensorMap ma, mb, md;
  bool ok = q8 ? make_q_map(&md, yq, N, M, ldq) : make_out_map(&md, y, N, M, ldy, false);
  ok = ok && make_map(&ma, xq, K, M, ldx, BM) && make_map(&mb, wq, K, N, ldw, 128);
  if (!ok) {
    cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return TWEO_ERR_CUDA;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = q8 ? smem5q : smem6;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (q8) TWEO_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern_q8, ma, mb, md, md, p));   // md doubles as the 8-bit output map
  else TWEO_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern_bf16, ma, mb, md, md, p));
  count_launch();
  return check_launch("gemm_fp8_pair_kernel (int8)");
}

}  // namespace tweo_detail

extern "C" {

tweo_status_t tweo_fp8_linear_fwd(const uint8_t* xq, int64_t ldx, const uint8_t* wq, int64_t ldw,
                                  const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                                  int64_t N, int64_t K, int32_t fmt_x, int32_t fmt_w, const tweo_epilogue_t* epi,
                                  void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_fp8_linear_fwd " "M=%lld N=%lld K=%lld fmt_x=%d fmt_w=%d ldx=%lld ldw=%lld ldy=%lld epi=%p ws=%p", (long long)M,(long long)N,(long long)K,fmt_x,fmt_w,(long long)ldx,(long long)ldw,(long long)ldy,(const void*)epi,ws);
  if (!xq || !wq || !sx_inv || !sw_inv || !y || !fmt_ok(fmt_x) || !fmt_ok(fmt_w)) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  return tweo_detail::gemm_fwd_codes(xq, ldx, fmt_x, wq, ldw, fmt_w, sx_inv, sw_inv, y, ldy, M, N, K, epi, ws,
                                     ws_bytes, (cudaStream_t)stream, false);
}

tweo_status_t tweo_fp8_linear_fwd_act(const uint8_t* xq, int64_t ldx, const uint8_t* wq, int64_t ldw,
                                      const float* sx_inv, const float* sw_inv, int32_t act, uint16_t* y, int64_t ldy,
                                      int64_t M, int64_t N, int64_t K, int32_t fmt_x, int32_t fmt_w,
                                      const tweo_epilogue_t* epi, void* stream) {
  TWEO_LOG_CALL("tweo_fp8_linear_fwd_act " "M=%lld N=%lld K=%lld act=%d fmt_x=%d fmt_w=%d epi=%p", (long long)M,(long long)N,(long long)K,act,fmt_x,fmt_w,(const void*)epi);
  if (act == TWEO_ACT_NONE)
    return tweo_fp8_linear_fwd(xq, ldx, wq, ldw, sx_inv, sw_inv, y, ldy, M, N, K, fmt_x, fmt_w, epi, nullptr, 0, stream);
  if (act != TWEO_ACT_GELU && act != TWEO_ACT_GELU_TANH && act != TWEO_ACT_SWIGLU) return TWEO_ERR_INVALID_ARG;
  if (!xq || !wq || !sx_inv || !sw_inv || !fmt_ok(fmt_x) || !fmt_ok(fmt_w)) return TWEO_ERR_INVALID_ARG;
  if (!y && !(epi && epi->out_q)) return TWEO_ERR_INVALID_ARG;  // nothing to write
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  GemmParams p{};
  p.d = y;
  p.ldd = y ? ldy : 0;
  p.sa_inv = sx_inv;
  p.sb_inv = sw_inv;
  tweo_status_t s = fill_epilogue(p, epi);
  if (s != TWEO_OK) return s;
  return run_fwd_act(xq, ldx, fmt_x, wq, ldw, fmt_w, false, act, M, N, K, p, (cudaStream_t)stream);
}

tweo_status_t tweo_fp8_linear_bwd_dgrad(const uint8_t* dyq, int64_t lddy, int32_t fmt_dy, const uint8_t* wq,
                                        int64_t ldw, int32_t fmt_w, const float* sdy_inv, const float* sw_inv,
                                        uint16_t* dx, int64_t lddx, int64_t M, int64_t N, int64_t K,
                                        const tweo_epilogue_t* epi, void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_fp8_linear_bwd_dgrad " "M=%lld N=%lld K=%lld fmt_dy=%d fmt_w=%d epi=%p ws=%p", (long long)M,(long long)N,(long long)K,fmt_dy,fmt_w,(const void*)epi,ws);
  if (!dyq || !wq || !sdy_inv || !sw_inv || !dx || !fmt_ok(fmt_dy) || !fmt_ok(fmt_w)) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  GemmParams p{};
  p.d = dx;
  p.ldd = lddx;
  p.sa_inv = sdy_inv;
  p.sb_inv = sw_inv;
  tweo_status_t s = fill_epilogue(p, epi);
  if (s != TWEO_OK) return s;
  // dX[M,K] = dYq[M,N] . Wq[N,K]: contraction over N; Wq is stored [N(contraction), K(out)] = MN-major
  if (epi && (epi->out_amax || epi->out_q) && M > 128 && K > 128)  // extra outputs leave through shared memory and TMA
    return run_fwd_act(dyq, lddy, fmt_dy, wq, ldw, fmt_w, true, TWEO_ACT_NONE, M, K, N, p, (cudaStream_t)stream);
  return run_gemm(Operand{dyq, lddy, fmt_dy, false}, Operand{wq, ldw, fmt_w, true}, M, K, N, p, ws, ws_bytes,
                  (cudaStream_t)stream);
}

tweo_status_t tweo_fp8_linear_bwd_wgrad(const uint8_t* xq, int64_t ldx, int32_t fmt_x, const uint8_t* dyq,
                                        int64_t lddy, int32_t fmt_dy, const float* sx_inv, const float* sdy_inv,
                                        void* dw, int64_t lddw, int32_t dw_dtype, int32_t accumulate, int64_t M,
                                        int64_t N, int64_t K, void* ws, size_t ws_bytes, void* stream) {
  TWEO_LOG_CALL("tweo_fp8_linear_bwd_wgrad " "M=%lld N=%lld K=%lld fmt_x=%d fmt_dy=%d ws=%p", (long long)M,(long long)N,(long long)K,fmt_x,fmt_dy,ws);
  if (!xq || !dyq || !sx_inv || !sdy_inv || !dw || !fmt_ok(fmt_x) || !fmt_ok(fmt_dy)) return TWEO_ERR_INVALID_ARG;
  if (dw_dtype != TWEO_BF16 && dw_dtype != TWEO_F32) return TWEO_ERR_INVALID_ARG;
  if (accumulate && dw_dtype != TWEO_F32) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  GemmParams p{};
  p.d = dw;
  p.ldd = lddw;
  p.sa_inv = sdy_inv;
  p.sb_inv = sx_inv;
  p.out_f32 = dw_dtype == TWEO_F32;
  p.accumulate = accumulate ? 1 : 0;
  fill_epilogue(p, nullptr);
  // dW[N,K] = dYq[M,N]^T . Xq[M,K]: contraction over M; both operands stored [M(contraction), out]
  return run_gemm(Operand{dyq, lddy, fmt_dy, true}, Operand{xq, ldx, fmt_x, true}, N, K, M, p, ws, ws_bytes,
                  (cudaStream_t)stream);
}

tweo_status_t tweo_fp8_linear_bwd(const uint8_t* dyq, int64_t lddy, int32_t fmt_dy, const uint8_t* xq, int64_t ldx,
                                  int32_t fmt_x, const uint8_t* wq, int64_t ldw, int32_t fmt_w, const float* sdy_inv,
                                  const float* sx_inv, const float* sw_inv, uint16_t* dx, int64_t lddx, uint16_t* dw,
                                  int64_t lddw, int64_t M, int64_t N, int64_t K, void* ws, size_t ws_bytes,
                                  void* stream) {
  TWEO_LOG_CALL("tweo_fp8_linear_bwd " "M=%lld N=%lld K=%lld fmt_dy=%d fmt_x=%d fmt_w=%d ws=%p", (long long)M,(long long)N,(long long)K,fmt_dy,fmt_x,fmt_w,ws);
  if (!dyq || !xq || !wq || !sdy_inv || !sx_inv || !sw_inv || !dx || !dw) return TWEO_ERR_INVALID_ARG;
  if (!fmt_ok(fmt_dy) || !fmt_ok(fmt_x) || !fmt_ok(fmt_w)) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!tweo_detail::aligned16(dyq) || !tweo_detail::aligned16(xq) || !tweo_detail::aligned16(wq) ||
      !tweo_detail::aligned16(dx) || !tweo_detail::aligned16(dw) || (lddy & 15) || (ldx & 15) || (ldw & 15) ||
      (lddx & 7) || (lddw & 7))
    return TWEO_ERR_ALIGNMENT;
  // both outputs large enough for 256 x 256 tiles: one launch; else the two products one after the other
  if (M > 128 && N > 128 && K > 128)
    return run_bwd_group(dyq, lddy, fmt_dy, xq, ldx, fmt_x, wq, ldw, fmt_w, sdy_inv, sx_inv, sw_inv, dx, lddx, dw, lddw,
                         M, N, K, (cudaStream_t)stream);
  tweo_status_t s = tweo_fp8_linear_bwd_dgrad(dyq, lddy, fmt_dy, wq, ldw, fmt_w, sdy_inv, sw_inv, dx, lddx, M, N, K,
                                              nullptr, ws, ws_bytes, stream);
  if (s != TWEO_OK) return s;
  return tweo_fp8_linear_bwd_wgrad(xq, ldx, fmt_x, dyq, lddy, fmt_dy, sx_inv, sdy_inv, dw, lddw, TWEO_BF16, 0, M, N, K,
                                   ws, ws_bytes, stream);
}

tweo_status_t tweo_fp8_linear_group(const tweo_linear_problem_t* problems, int32_t count, void* stream) {
  TWEO_LOG_CALL("tweo_fp8_linear_group " "problems=%p count=%d", (const void*)problems, count);
  if (!problems || count < 1 || count > TWEO_MAX_GROUP) return TWEO_ERR_INVALID_ARG;
  GroupDesc d[TWEO_MAX_GROUP];
  for (int i = 0; i < count; ++i) {
    const tweo_linear_problem_t& q = problems[i];
    const int64_t M = q.M, N = q.N, K = q.K;
    if (!q.out || M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
    if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
    if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return TWEO_ERR_UNSUPPORTED_SHAPE;
    if (!tweo_detail::aligned16(q.out) || (q.ldo & 7)) return TWEO_ERR_ALIGNMENT;
    switch (q.product) {
      case TWEO_PRODUCT_FWD:    // Y[M,N] = Xq[M,K] . Wq[N,K]^T
        if (!q.xq || !q.wq || !q.sx_inv || !q.sw_inv || !fmt_ok(q.fmt_x) || !fmt_ok(q.fmt_w)) return TWEO_ERR_INVALID_ARG;
        d[i] = GroupDesc{q.xq, q.wq, q.ldx, q.ldw, M, N, K, q.fmt_x, q.fmt_w, false, false, q.out, q.ldo, q.sx_inv, q.sw_inv};
        break;
      case TWEO_PRODUCT_DGRAD:  // dX[M,K] = dYq[M,N] . Wq[N,K]
        if (!q.dyq || !q.wq || !q.sdy_inv || !q.sw_inv || !fmt_ok(q.fmt_dy) || !fmt_ok(q.fmt_w)) return TWEO_ERR_INVALID_ARG;
        d[i] = GroupDesc{q.dyq, q.wq, q.lddy, q.ldw, M, K, N, q.fmt_dy, q.fmt_w, false, true, q.out, q.ldo, q.sdy_inv, q.sw_inv};
        break;
      case TWEO_PRODUCT_WGRAD:  // dW[N,K] = dYq[M,N]^T . Xq[M,K]
        if (!q.dyq || !q.xq || !q.sdy_inv || !q.sx_inv || !fmt_ok(q.fmt_dy) || !fmt_ok(q.fmt_x)) return TWEO_ERR_INVALID_ARG;
        d[i] = GroupDesc{q.dyq, q.xq, q.lddy, q.ldx, N, K, M, q.fmt_dy, q.fmt_x, true, true, q.out, q.ldo, q.sdy_inv, q.sx_inv};
        break;
      default:
        return TWEO_ERR_INVALID_ARG;
    }
    if (q.epi && (q.epi->out_amax || q.epi->out_q)) {
      if (q.product == TWEO_PRODUCT_WGRAD) return TWEO_ERR_INVALID_ARG;   // the fused outputs feed the next linear: Y and dX only
      d[i].out_amax = q.epi->out_amax;
      if (q.epi->out_q) {
        if (!q.epi->q_scale || !fmt_ok(q.epi->q_fmt)) return TWEO_ERR_INVALID_ARG;
        if (!tweo_detail::aligned16(q.epi->out_q) || (q.epi->ldq & 15)) return TWEO_ERR_ALIGNMENT;
        d[i].out_q = q.epi->out_q;
        d[i].ldq = q.epi->ldq;
        d[i].q_fmt = q.epi->q_fmt;
        d[i].q_scale = q.epi->q_scale;
      }
    }
    if (d[i].Md <= 128 || d[i].Nd <= 128) return TWEO_ERR_UNSUPPORTED_SHAPE;   // the pair kernel's 256 x 256 tiles
    if (!tweo_detail::aligned16(d[i].a) || !tweo_detail::aligned16(d[i].b) || (d[i].lda & 15) || (d[i].ldb & 15))
      return TWEO_ERR_ALIGNMENT;
  }
  return run_group(d, count, (cudaStream_t)stream);
}

tweo_status_t tweo_fp4_weight_linear(const uint8_t* xq, int64_t ldx, int32_t fmt_x, const float* sx_inv, const uint8_t* w4,
                                     int64_t ldw_bytes, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M, int64_t N,
                                     int64_t K, void* stream) {
  TWEO_LOG_CALL("tweo_fp4_weight_linear " "M=%lld N=%lld K=%lld fmt_x=%d ldx=%lld ldw_bytes=%lld", (long long)M,(long long)N,(long long)K,fmt_x,(long long)ldx,(long long)ldw_bytes);
  if (!xq || !sx_inv || !w4 || !sw_inv || !y || !fmt_ok(fmt_x)) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if (M > 128 || (N & 15) || (K & 127)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  if (!tweo_detail::aligned16(y) || (ldy & 7)) return TWEO_ERR_ALIGNMENT;
  return run_skinny_w4(xq, ldx, fmt_x, w4, ldw_bytes, sx_inv, sw_inv, y, ldy, M, N, K, (cudaStream_t)stream);
}

tweo_status_t tweo_selftest_bounded_wait(uint64_t limit_ns, uint32_t* gave_up, void* stream) {
  if (limit_ns < 1000ull || limit_ns > 100000000ull) return TWEO_ERR_INVALID_ARG;  // 1 us .. 100 ms
  bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_ns, gave_up);
  tweo_detail::count_launch();
  return tweo_detail::check_launch("bounded_wait_selftest_kernel");
}

tweo_status_t tweo_int8_linear(const int8_t* xq, int64_t ldx, const float* sx, int32_t sx_per_row, const int8_t* wq,
                               int64_t ldw, const float* sw, int32_t sw_per_row, int32_t bits, uint16_t* y, int64_t ldy,
                               int64_t M, int64_t N, int64_t K, void* stream) {
  TWEO_LOG_CALL("tweo_int8_linear " "M=%lld N=%lld K=%lld bits=%d sx_per_row=%d sw_per_row=%d", (long long)M,(long long)N,(long long)K,bits,sx_per_row,sw_per_row);
  if (!y) return TWEO_ERR_INVALID_ARG;
  return tweo_detail::run_int8_linear(xq, ldx, sx, sx_per_row, wq, ldw, sw, sw_per_row, bits, y, ldy, nullptr, 0,
                                      nullptr, M, N, K, (cudaStream_t)stream);
}

tweo_status_t tweo_int8_linear_q8(const int8_t* xq, int64_t ldx, const float* sx, int32_t sx_per_row, const int8_t* wq,
                                  int64_t ldw, const float* sw, int32_t sw_per_row, int32_t bits, const float* sy,
                                  int8_t* yq, int64_t ldq, int64_t M, int64_t N, int64_t K, void* stream) {
  TWEO_LOG_CALL("tweo_int8_linear_q8 " "M=%lld N=%lld K=%lld bits=%d sx_per_row=%d sw_per_row=%d ldq=%lld", (long long)M,(long long)N,(long long)K,bits,sx_per_row,sw_per_row,(long long)ldq);
  if (!yq || !sy) return TWEO_ERR_INVALID_ARG;
  return tweo_detail::run_int8_linear(xq, ldx, sx, sx_per_row, wq, ldw, sw, sw_per_row, bits, nullptr, 0, yq, ldq, sy,
                                      M, N, K, (cudaStream_t)stream);
}

}  // extern "C"
