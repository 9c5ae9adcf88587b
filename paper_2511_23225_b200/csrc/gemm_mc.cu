// Optional accelerator library for the CTA-pair FP8 GEMM: clusters of FOUR CTAs (two pairs that
// compute vertically adjacent 256 x 256 tiles and therefore read the same B tile).  Every CTA
// fetches only half of its B half from L2 and the TMA unit delivers it to the CTA of the same
// parity in both pairs (cluster multicast), so an SM pulls 24 KB per 128-deep contraction
// block instead of 32 KB.  The L2 -> shared-memory path is what limits the two-CTA kernel on
// large tensor-bound shapes, so this is where the remaining headroom is.
//
// All operands are this GPU's own memory.  The file is built into a library of its own
// (libtweo_b200_mc.so) that the main library loads if it is there; everything works without
// it.  It is meant for single-GPU runs only and is left out of multi-GPU deployments.
#include <cuda.h>
#include <cuda_runtime.h>

#include "gemm_common.cuh"
#include "gemm_pair.cuh"
#include "tc_ptx.cuh"

namespace {

using namespace tweo_detail;

struct PairCfgMc {
  static constexpr int kPairs = 2;
  // This CTA's half of the B tile is 128 rows x 128 bytes; pair `pr` of the cluster fetches rows
  // [64 pr, 64 pr + 64) of it and multicasts them to the CTAs of its own parity in both pairs.
  // The completion is signalled on the full barrier of each receiving CTA's pair leader (same
  // CTA-relative offset; clearing bit 24 of the shared-window address selects the even CTA).
  static __device__ __forceinline__ void load_b(uint32_t sb, const CUtensorMap* map, int32_t c0, int32_t c1,
                                                bool b_mn, uint32_t lead_bar, uint32_t local_bar, uint32_t crank) {
    (void)b_mn;
    (void)lead_bar;
    const uint32_t pr = crank >> 1, parity = crank & 1u;
    const uint16_t mask = (uint16_t)((1u << parity) | (1u << (2u + parity)));
    const uint32_t dst = sb + pr * (64u * 128u);
    const uint32_t bar = local_bar & 0xFEFFFFFFu;
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1 + (int32_t)(64u * pr)), "r"(bar), "h"(mask)
        : "memory");
  }
};

constexpr int kStages = 6;
constexpr size_t kSmem = (size_t)kStages * (BM * BK + 128 * BK) + 4 * 2 * 32 * 128 + 1024 + 256;

template <bool A_MN, bool B_MN, bool OUT_F32>
cudaError_t launch(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, GemmParams p, cudaStream_t st) {
  auto kern = gemm_fp8_pair_kernel<PairCfgMc, A_MN, B_MN, kStages, OUT_F32>;
  static int max_clusters = -1;  // per instantiation; all instantiations have the same footprint
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 4;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_clusters < 0) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
    if (e != cudaSuccess) return e;
    int n = 0;
    cfg.gridDim = dim3(4u * 64u);
    e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (n < 1) return cudaErrorInvalidConfiguration;
    max_clusters = n;
  }
  p.tiles_m = (p.Md + 4 * BM - 1) / (4 * BM);  // super-tiles of 512 rows
  p.tiles_n = (p.Nd + 255) / 256;
  p.k_blocks = (p.Kc + BK - 1) / BK;
  p.sk_tiles = 0;
  p.sk_partials = nullptr;
  p.sk_flags = nullptr;
  p.sk_counters = nullptr;
  const int tiles = p.tiles_m * p.tiles_n;
  int clusters = max_clusters < tiles ? max_clusters : tiles;
  p.raster_g = raster_band(p.tiles_m, max_clusters);
  cfg.gridDim = dim3((unsigned)(4 * clusters));
  return cudaLaunchKernelEx(&cfg, kern, ma, mb, md, p);
}

}  // namespace

extern "C" {

// Launches D = A . B with the four-CTA-cluster kernel.  `mb` must be a tensor map of B with boxes
// of 128 bytes x 64 rows.  Returns a cudaError_t value.
__attribute__((visibility("default"))) int tweo_mc_gemm(const CUtensorMap* ma, const CUtensorMap* mb,
                                                        const CUtensorMap* md, const GemmParams* p, int a_mn, int b_mn,
                                                        void* stream) {
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (!a_mn && !b_mn) e = p->out_f32 ? launch<false, false, true>(*ma, *mb, *md, *p, st) : launch<false, false, false>(*ma, *mb, *md, *p, st);
  else if (!a_mn && b_mn) e = p->out_f32 ? launch<false, true, true>(*ma, *mb, *md, *p, st) : launch<false, true, false>(*ma, *mb, *md, *p, st);
  else if (a_mn && b_mn) e = p->out_f32 ? launch<true, true, true>(*ma, *mb, *md, *p, st) : launch<true, true, false>(*ma, *mb, *md, *p, st);
  else return (int)cudaErrorInvalidValue;
  if (e == cudaSuccess) e = cudaGetLastError();
  return (int)e;
}

// Reads and clears this library's record of expired device-side waits (0 = none).
__attribute__((visibility("default"))) int tweo_mc_read_status(unsigned int* out) {
  unsigned int v = 0, zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&v, g_device_status, sizeof v);
  if (e != cudaSuccess) return (int)e;
  if (v != 0) e = cudaMemcpyToSymbol(g_device_status, &zero, sizeof zero);
  *out = v;
  return (int)e;
}

}  // extern "C"
