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
// are split evenly over all CTAs.  A CTA whose share starts in the middle of a tile writes
// its raw fp32 accumulator to a workspace slot and raises a flag; the CTA that owns the
// tile's first k-block adds the other shares in CTA order (fixed order => reproducible)
// and runs the epilogue.  Such a share is always the FIRST thing a CTA does and an owner's
// wait is the LAST step of its stream-K work, so waits cannot form a cycle.
//
// Every wait (mbarrier or flag) is bounded: on expiry the CTA records TWEO_ERR_TIMEOUT in
// a device status word, drains and exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <cstdlib>
#include <mutex>

#include "common.cuh"

namespace {

using namespace tweo_detail;

constexpr int BM = 128;      // rows of D per tile = tcgen05 M (lanes of tensor memory)
constexpr int BK = 128;      // contraction bytes per stage = one 128-byte swizzle span
constexpr int UMMA_K = 32;   // contraction per instruction for 8-bit operands
constexpr int kThreads = 192;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s

__device__ unsigned int g_device_status = 0;

struct GemmParams {
  void* d;
  int64_t ldd;
  int32_t Md, Nd, Kc;
  int32_t tiles_m, tiles_n, k_blocks;
  int32_t raster_g;    // tiles are numbered in bands of raster_g tile rows (see tile_coords)
  const float* sa_inv;
  const float* sb_inv;
  int32_t out_f32;     // 0: bf16 out, 1: fp32 out
  int32_t accumulate;  // fp32 out only
  float* out_amax;
  uint8_t* out_q;
  int64_t ldq;
  int32_t q_fmt;
  const float* q_scale;
  uint32_t idesc;
  // stream-K: tiles [0, sk_tiles) are split along the contraction, the rest dealt whole
  int32_t sk_tiles;
  float* sk_partials;   // [grid][BM*BN] raw accumulators of shares that do not own their tile
  uint32_t* sk_flags;   // [grid][4] per epilogue warp: == epoch once the share is written
  uint32_t* sk_counters;  // CTA-pair kernel: [sk_tiles][2][4] tickets per (tile, CTA of the pair, epilogue warp)
  uint32_t epoch;
};

// Workspace layout of the linear calls (bytes from the workspace base):
//   [0, 4096)       flags of the single-CTA kernel's split tiles (4 words per CTA)
//   [4096, 12288)   ticket counters of the CTA-pair kernel's split tiles (8 words per tile)
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

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* ptr) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* ptr, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}

// ----------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: false if the CTA is aborting or the limit expired (then it raises abort).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 0x3FFu) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(&g_device_status, (unsigned int)TWEO_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

// shared -> global tile store (bulk async group); out-of-range rows / columns are clipped
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
// same, but adds the tile to what global memory holds (fp32 accumulate)
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t src) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem] (+)= A[smem] . B[smem]
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i gets row (lane base + i), columns c..c+31
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  Fields (bit positions):
//   [0,14)  start address >> 4        [16,30) leading-dimension byte offset >> 4
//   [32,46) stride byte offset >> 4   [46,48) descriptor version = 1 (sm_100)
//   [61,64) swizzle mode, 2 = 128 B
// K-major tile: rows of 128 contraction bytes, 8-row groups 1024 B apart (stride offset);
//   the leading offset is unused for swizzled K-major layouts.
// MN-major tile: rows are contraction indices holding 128 contiguous bytes of the output
//   dimension; 8-row groups 1024 B apart (stride offset); further 128-wide slabs of the
//   output dimension `slab_bytes` apart (leading offset).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// ----------------------------------------------------------------- epilogue helpers
template <int FMT>
__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d) {
  return cvt_fp8x2<FMT>(a, b) | (cvt_fp8x2<FMT>(c, d) << 16);
}

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
    const float alpha = __fmul_rn(__ldg(p.sa_inv), __ldg(p.sb_inv));
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
      if (kb0 > 0) {
        // A share that does not own its tile: park the raw accumulator, raise the flag.
        float* slot = p.sk_partials + (size_t)blockIdx.x * (BM * BN);
#pragma unroll 1
        for (int g = 0; g < BN / 32; ++g) {
          uint32_t r[32];
          tmem_ld32(tmem_base + tlane + (uint32_t)(acc * BN + g * 32), r);
          tmem_ld_wait();
          float* dst = slot + ((g * 4 + quarter) * 32) * 32 + lane;
#pragma unroll
          for (int k = 0; k < 32; ++k) __stcg(dst + k * 32, __uint_as_float(r[k]));
        }
        __threadfence();
        __syncwarp();
        if (lane == 0) st_release_u32(p.sk_flags + blockIdx.x * 4 + quarter, p.epoch);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        continue;
      }
      int n_contrib = 0;
      if (kb1 < p.k_blocks) {
        // Owner of a tile whose later k-blocks went to the following CTAs: wait for them.
        const int64_t tile_end = (int64_t)(tile + 1) * p.k_blocks;
        for (int j = blockIdx.x + 1; j < (int)gridDim.x && Sched::share_begin(p, j, gridDim.x) < tile_end; ++j) {
          const uint32_t* flag = p.sk_flags + j * 4 + quarter;
          if (ld_acquire_u32(flag) != p.epoch) {
            const uint64_t t0 = globaltimer_ns();
            for (uint32_t spin = 1; ld_acquire_u32(flag) != p.epoch; ++spin) {
              if ((spin & 0xFFu) == 0) {
                if (*abort_flag) { ok = false; break; }
                if (globaltimer_ns() - t0 > kWaitLimitNs) {
                  *abort_flag = 1;
                  atomicExch(&g_device_status, (unsigned int)TWEO_ERR_TIMEOUT);
                  ok = false;
                  break;
                }
              }
            }
          }
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          ++n_contrib;
        }
        if (!ok) break;
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
        for (int jc = 0; jc < n_contrib; ++jc) {  // add the other shares, in CTA order
          const float* part = p.sk_partials + (size_t)(blockIdx.x + 1 + jc) * (BM * BN);
#pragma unroll
          for (int h = 0; h < CH / 32; ++h) {
            const float* src = part + (((c * (CH / 32) + h) * 4 + quarter) * 32) * 32 + lane;
#pragma unroll
            for (int k = 0; k < 32; ++k)
              r[h * 32 + k] = __float_as_uint(__uint_as_float(r[h * 32 + k]) + __ldcg(src + k * 32));
          }
        }
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


// ----------------------------------------------------------------- CTA-pair kernel
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
//   tempty[a]  leader only : 4 epilogue warps of each CTA arrive (the peer's remotely)
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1,
                                                 uint32_t leader_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(leader_bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_f8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives (at the given cluster-window address) once all MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t cluster_bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar)
               : "memory");
}

// A share of the pair kernel that covers only part of a split tile.  Parks this warp's
// 32 x 256 block of the raw accumulator in the workspace ([column][row], so every store is
// one full line), hands the accumulator back to the MMA warp and takes a ticket; the warp
// that draws the last ticket of the tile adds the parked blocks of ALL shares in share order
// (= ascending k, whoever arrived last, so the sum does not depend on timing) and stores the
// result.  Nobody waits for anybody.  Kept out of line: it is rare and register-hungry.
constexpr size_t kPairCtaFloats = 128 * 256;   // one CTA's half of a parked 256 x 256 accumulator
constexpr size_t kPairWarpFloats = 32 * 256;   // one epilogue warp's block of it

template <bool OUT_F32>
__device__ __noinline__ float pair_partial_share(const GemmParams& p, const CUtensorMap* tmap_d, int tile, int kb0,
                                                int pair, int num_pairs, int rank, int wslot,
                                                uint32_t tacc, uint32_t tempty_leader, float alpha, float qs,
                                                uint32_t epi_base, uint32_t it, int lane, int row0, int n0) {
  constexpr int CH = OUT_F32 ? 32 : 64;
  constexpr uint32_t EPI_BUF = 32 * 128;
  float run_amax = 0.0f;
  float* slot = p.sk_partials + ((size_t)(pair * 2 + (kb0 > 0 ? 0 : 1)) * 2 + rank) * kPairCtaFloats +
                (size_t)wslot * kPairWarpFloats;
#pragma unroll 1
  for (int g = 0; g < 8; ++g) {
    uint32_t r[32];
    tmem_ld32(tacc + (uint32_t)(g * 32), r);
    tmem_ld_wait();
    float* dst = slot + g * 1024 + lane;
#pragma unroll
    for (int k = 0; k < 32; ++k) __stcg(dst + k * 32, __uint_as_float(r[k]));
  }
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive_cluster(tempty_leader);
  // which pairs hold a share of this tile (they are consecutive)
  const int64_t t_begin = (int64_t)tile * p.k_blocks, t_end = t_begin + p.k_blocks;
  int j_first = pair;
  while (j_first > 0 && Sched::share_begin(p, j_first, num_pairs) > t_begin) --j_first;
  int j_last = pair;
  while (j_last + 1 < num_pairs && Sched::share_begin(p, j_last + 1, num_pairs) < t_end) ++j_last;
  const int n_shares = j_last - j_first + 1;
  __threadfence();
  __syncwarp();
  uint32_t ticket = 0;
  uint32_t* counter = p.sk_counters + ((size_t)tile * 2 + rank) * 4 + wslot;
  if (lane == 0) ticket = atomicAdd(counter, 1u);
  ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
  if (ticket + 1 != (uint32_t)n_shares) return 0.0f;  // not the last share of this tile: done
  __threadfence();
  if (lane == 0) *counter = 0u;  // ready for the next launch
  const uint32_t row_off = (uint32_t)lane * 128u;
  const uint32_t swz = (uint32_t)(lane & 7);
  const int row = row0 + lane;
#pragma unroll 1
  for (int c = 0; c < 256 / CH; ++c) {
    const int col0 = n0 + c * CH;
    if (col0 >= p.Nd || row0 >= p.Md) break;  // uniform across the warp
    uint32_t r[CH];
#pragma unroll 1
    for (int sidx = 0; sidx < n_shares; ++sidx) {
      const int j = j_first + sidx;
      const int sel = Sched::share_begin(p, j, num_pairs) > t_begin ? 0 : 1;
      const float* src = p.sk_partials + ((size_t)(j * 2 + sel) * 2 + rank) * kPairCtaFloats +
                         (size_t)wslot * kPairWarpFloats + (size_t)(c * CH) * 32 + lane;
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
      if ((p.out_amax || p.out_q) && row < p.Md) {
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

template <bool A_MN, bool B_MN, int STAGES, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_fp8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_d, const __grid_constant__ GemmParams p) {
  constexpr int BN = 256;                 // tile columns of the pair
  constexpr uint32_t A_BYTES = BM * BK;   // this CTA's 128 rows of A
  constexpr uint32_t B_BYTES = 128 * BK;  // this CTA's 128 of the 256 columns of B
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 512;

  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  constexpr uint32_t EPI_BUF = 32 * 128;
  constexpr uint32_t EPI_BYTES = 4 * 2 * EPI_BUF;
  uint8_t* epi_smem = smem + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_smem + EPI_BYTES);
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
      mbar_init(tempty_bar(a), 8);  // four epilogue warps of each CTA of the pair
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

  const int pair = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      Sched sched(p, pair, num_pairs);
      int tile, kb0, kb1;
      while (ok && sched.next(tile, kb0, kb1)) {
        int tm, tn;
        tile_coords(p, tile, tm, tn);
        const int m0 = tm * (2 * BM) + (int)rank * BM;  // this CTA's rows
        const int n0 = tn * BN + (int)rank * 128;       // this CTA's half of B
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          const int k0 = kb * BK;
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
      Sched sched(p, pair, num_pairs);
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
            const uint64_t adesc = make_smem_desc(sa + (A_MN ? k * UMMA_K * 128 : k * UMMA_K), BK * 128);
            const uint64_t bdesc = make_smem_desc(sb + (B_MN ? k * UMMA_K * 128 : k * UMMA_K), BK * 128);
            umma_f8_pair(d_tmem, adesc, bdesc, p.idesc, (uint32_t)(kb != kb0 || k != 0));
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
    // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int quarter = warp & 3;
    const float alpha = __fmul_rn(__ldg(p.sa_inv), __ldg(p.sb_inv));
    const float qs = p.out_q ? __ldg(p.q_scale) : 0.0f;
    constexpr int CH = OUT_F32 ? 32 : 64;
    const uint32_t epi_base = smem_u32(epi_smem) + (uint32_t)(warp - 2) * 2u * EPI_BUF;
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t swz = (uint32_t)(lane & 7);
    const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
    uint32_t it = 0;
    float run_amax = 0.0f;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    Sched sched(p, pair, num_pairs);
    int tile, kb0, kb1;
    while (ok && sched.next(tile, kb0, kb1)) {
      int tm, tn;
      tile_coords(p, tile, tm, tn);
      const int m0 = tm * (2 * BM) + (int)rank * BM;
      const int n0 = tn * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row0 = m0 + quarter * 32;
      const int row = row0 + lane;
      const bool row_ok = row < p.Md;
      if (kb0 != 0 || kb1 != p.k_blocks) {
        // part of a split tile: park the accumulator; the last share to arrive stores the tile
        const float part_amax = pair_partial_share<OUT_F32>(
            p, &tmap_d, tile, kb0, pair, num_pairs, (int)rank, warp - 2,
            tmem_base + tlane + (uint32_t)(acc * BN), map_to_cta(tempty_bar(acc), 0), alpha, qs, epi_base, it, lane,
            row0, n0);
        it += BN / CH;  // keeps the staging-buffer rotation in step whether or not this warp stored
        run_amax = fmaxf(run_amax, part_amax);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        continue;
      }
#pragma unroll 1
      for (int c = 0; c < BN / CH; ++c) {
        const int col0 = n0 + c * CH;
        if (col0 >= p.Nd) break;
        uint32_t r[CH];
        const uint32_t taddr = tmem_base + tlane + (uint32_t)(acc * BN + c * CH);
        tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        if (!OUT_F32) tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[CH - 32]));
        tmem_ld_wait();
        if (row0 >= p.Md) continue;
        const uint32_t buf = epi_base + (it & 1u) * EPI_BUF;
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
#pragma unroll
            for (int h = 0; h < 2; ++h) {
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
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));  // the leader's barrier
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (lane == 0) bulk_wait_all();
    if (p.out_amax) {
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

__global__ void zero_float_kernel(float* p) { *p = 0.0f; }

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

uint32_t make_idesc(int fmt_a, int fmt_b, bool a_mn, bool b_mn, int n, int m = BM) {
  // [4,6) accumulator format (1 = fp32)   [7,10) A format   [10,13) B format (0 = E4M3, 1 = E5M2)
  // [15] A major (1 = MN)   [16] B major   [17,23) N >> 3   [24,29) M >> 4
  uint32_t d = 0;
  d |= 1u << 4;
  d |= (uint32_t)(fmt_a == TWEO_E5M2 ? 1 : 0) << 7;
  d |= (uint32_t)(fmt_b == TWEO_E5M2 ? 1 : 0) << 10;
  d |= (uint32_t)(a_mn ? 1 : 0) << 15;
  d |= (uint32_t)(b_mn ? 1 : 0) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(m >> 4) << 24;
  return d;
}

std::atomic<uint32_t> g_sk_epoch{0};
// TWEO_GEMM_NO_PAIR=1 in the environment keeps every GEMM on the single-CTA kernel (A/B timing).
const bool g_disable_pair = [] { const char* e = getenv("TWEO_GEMM_NO_PAIR"); return e && e[0] == '1'; }();

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
  static bool attr_done = false;  // per instantiation
  if (!attr_done) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attr_done = true;
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
  p.sk_flags = nullptr;
  p.sk_counters = nullptr;
  p.epoch = 0;
  // Stream-K when whole-tile dealing would idle more than ~15 % of the SM-time and the
  // contraction is long enough to pay for the fix-up (a 128 x BN fp32 round trip through L2).
  const size_t sk_need = kWsPartialsOffset + (size_t)sms * kWsPartialBytesPerSm;
  const int waves = (tiles + sms - 1) / sms;
  if (ws && ws_bytes >= sk_need && aligned16(ws) && p.k_blocks >= 12 &&
      (double)tiles < 0.85 * (double)waves * sms) {
    const int full = tiles / sms;
    p.sk_tiles = full == 0 ? tiles : tiles - (full - 1) * sms;
    grid = sms;
    if ((int64_t)p.sk_tiles * p.k_blocks < grid) grid = (int)((int64_t)p.sk_tiles * p.k_blocks);
    p.sk_flags = reinterpret_cast<uint32_t*>(ws);
    p.sk_partials = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + kWsPartialsOffset);
    p.epoch = g_sk_epoch.fetch_add(1, std::memory_order_relaxed) + 1;
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
  auto kern = gemm_fp8_pair_kernel<A_MN, B_MN, STAGES, OUT_F32>;
  static bool attr_done = false;
  if (!attr_done) {
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    TWEO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 0));
    attr_done = true;
  }
  p.tiles_m = (p.Md + 2 * BM - 1) / (2 * BM);
  p.tiles_n = (p.Nd + 255) / 256;
  p.k_blocks = (p.Kc + BK - 1) / BK;
  p.sk_tiles = 0;
  p.sk_partials = nullptr;
  p.sk_flags = nullptr;
  p.sk_counters = nullptr;
  p.epoch = 0;
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
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  TWEO_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, ma, mb, md, p));
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
  const bool use_pair = Md > 128 && Nd > 128 && !g_disable_pair;
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
    zero_float_kernel<<<1, 1, 0, st>>>(p.out_amax);
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
                             cudaStream_t st) {
  GemmParams p{};
  p.d = y;
  p.ldd = ldy;
  p.sa_inv = sx_inv;
  p.sb_inv = sw_inv;
  tweo_status_t s = fill_epilogue(p, epi);
  if (s != TWEO_OK) return s;
  return run_gemm(Operand{xq, ldx, fmt_x, false}, Operand{wq, ldw, fmt_w, false}, M, N, K, p, ws, ws_bytes, st);
}

}  // namespace tweo_detail

extern "C" {

tweo_status_t tweo_fp8_linear_fwd(const uint8_t* xq, int64_t ldx, const uint8_t* wq, int64_t ldw,
                                  const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                                  int64_t N, int64_t K, int32_t fmt_x, int32_t fmt_w, const tweo_epilogue_t* epi,
                                  void* ws, size_t ws_bytes, void* stream) {
  if (!xq || !wq || !sx_inv || !sw_inv || !y || !fmt_ok(fmt_x) || !fmt_ok(fmt_w)) return TWEO_ERR_INVALID_ARG;
  if (M < 1 || N < 1 || K < 1) return TWEO_ERR_INVALID_ARG;
  if ((N & 15) || (K & 15)) return TWEO_ERR_UNSUPPORTED_SHAPE;
  return tweo_detail::gemm_fwd_codes(xq, ldx, fmt_x, wq, ldw, fmt_w, sx_inv, sw_inv, y, ldy, M, N, K, epi, ws,
                                     ws_bytes, (cudaStream_t)stream);
}

tweo_status_t tweo_fp8_linear_bwd_dgrad(const uint8_t* dyq, int64_t lddy, int32_t fmt_dy, const uint8_t* wq,
                                        int64_t ldw, int32_t fmt_w, const float* sdy_inv, const float* sw_inv,
                                        uint16_t* dx, int64_t lddx, int64_t M, int64_t N, int64_t K,
                                        const tweo_epilogue_t* epi, void* ws, size_t ws_bytes, void* stream) {
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
  return run_gemm(Operand{dyq, lddy, fmt_dy, false}, Operand{wq, ldw, fmt_w, true}, M, K, N, p, ws, ws_bytes,
                  (cudaStream_t)stream);
}

tweo_status_t tweo_fp8_linear_bwd_wgrad(const uint8_t* xq, int64_t ldx, int32_t fmt_x, const uint8_t* dyq,
                                        int64_t lddy, int32_t fmt_dy, const float* sx_inv, const float* sdy_inv,
                                        void* dw, int64_t lddw, int32_t dw_dtype, int32_t accumulate, int64_t M,
                                        int64_t N, int64_t K, void* ws, size_t ws_bytes, void* stream) {
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

}  // extern "C"
