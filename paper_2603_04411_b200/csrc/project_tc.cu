// Projection to the spectral space on the 5th-generation tensor cores:  X~ = X U  (Eq. 1), for the
// pre-RoPE key and value states of a batch of tokens, result rounded once to the 16-bit storage type.
//
// Work item = (128-token tile, side K or V, slab of NS output columns); NS = 256, or 128 when d is not a
// multiple of 256.  Items are dealt round-robin to one persistent CTA per SM, the slabs of one tile
// next to each other, so neighbouring CTAs read the same token tile from L2 at about the same time and
// a call of a few tokens still spreads over 2 d / NS CTAs.
// Per item the [128 x NS] fp32 accumulator is built by tcgen05.mma chains (M = 128, N = NS, K = 16 per
// instruction) in one of two alternating TMEM buffers; [128 x 64] panels of X and [NS x 64] panels of
// U^T (pre-transposed once, so it is the K-major B operand) stream through a 4-stage TMA ring with the
// 128-byte swizzle.  Epilogue warps read the accumulator with tcgen05.ld, round to f16 / bf16, write
// [128 x 64] panels into shared memory in the swizzled layout and hand them to TMA stores, which also
// clip the rows past the last token.
//
// Warp roles (320 threads):
//   warp 0      TMA producer: lanes 0-3 the U^T panel of ring stage L, lanes 4-7 the X panel of stage L - 4
//   warp 1      MMA issuer (one elected lane; owns the TMEM allocation)
//   warps 2-9   epilogue: thread = one token row x half of the slab's columns; each half (four warps) owns
//               one staging panel and one lane that issues its stores
// Calls of at least 1024 tokens with d a multiple of 256 run the CTA-pair variant further down instead.
// All barrier waits are bounded (tc_util.cuh); a wait that runs out ends the kernel with TWKV_ERR_TIMEOUT.
#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {
using namespace tc;

constexpr int PJ_THREADS = 320;
constexpr int PJ_EPI = 256;
constexpr int PJ_STAGES = 4;
constexpr uint32_t PJ_TMEM_COLS = 512;
constexpr uint32_t PJ_PANEL_BYTES = 16384;                      // [128 rows][64 x 16 bit]

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the stores committed by this thread have finished reading shared memory
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... and have been written out
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Barrier over `threads` threads that also ANDs a predicate across them.
__device__ __forceinline__ bool named_bar_and(int id, int threads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred), "r"(id), "r"(threads) : "memory");
  return r != 0;
}
__device__ __forceinline__ uint32_t pack_f16x2_rn(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

__global__ void __launch_bounds__(PJ_THREADS, 1)
project_tc_kernel(const __grid_constant__ CUtensorMap map_xk, const __grid_constant__ CUtensorMap map_xv,
                  const __grid_constant__ CUtensorMap map_uk, const __grid_constant__ CUtensorMap map_uv,
                  const __grid_constant__ CUtensorMap map_ok, const __grid_constant__ CUtensorMap map_ov,
                  int n_tok, int d, int bf16, int side0, int n_sides, int* status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int KP = d / PANEL;
  const int NS = (d % 256 == 0) ? 256 : 128;
  const int n_slabs = d / NS;
  const uint32_t b_stage_bytes = (uint32_t)NS * 128u;
  const uint32_t stage_bytes = PJ_PANEL_BYTES + b_stage_bytes;           // [X panel | U^T panel]
  const uint32_t sA = smem_addr(smem_raw);
  if (sA & 1023u) {
    if (tid == 0) atomicCAS(status, 0, TWKV_ERR_DEVICE_CHECK);
    return;
  }
  unsigned char* out_stage = smem_raw + PJ_STAGES * stage_bytes;         // two output panels, one per column half
  unsigned char* tail = out_stage + 2 * PJ_PANEL_BYTES;
  const uint32_t bars = smem_addr(tail);
  const uint32_t full = bars, empty = full + 8 * PJ_STAGES, acc_full = empty + 8 * PJ_STAGES, acc_empty = acc_full + 16;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (2 * PJ_STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  if (tid == 0) {
    for (int i = 0; i < PJ_STAGES; ++i) { mbar_init(full + 8 * i, 1); mbar_init(empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, PJ_EPI / 32); }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(smem_addr(s_tmem_base), PJ_TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // item -> (tile, side, slab): slab fastest, then side
  const int per_tile = n_sides * n_slabs;
  const int n_items = per_tile * ((n_tok + TILE - 1) / TILE);
  const int it0 = blockIdx.x, itstep = gridDim.x;
  const uint32_t n_acc = it0 < n_items ? (uint32_t)((n_items - it0 + itstep - 1) / itstep) : 0u;      // one accumulator per item

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    // one elected thread issues every copy in ring order: a copy issued from a lane picked by its index costs the warp
    // hundreds of cycles, and lanes of one warp that wait on different barriers wait one after the other
    if (elect_one()) {
      tma_prefetch_desc(&map_uk); tma_prefetch_desc(&map_uv);
      tma_prefetch_desc(&map_xk); tma_prefetch_desc(&map_xv);
      ring_gemm_produce<1>(n_acc, KP, PJ_STAGES, sA, stage_bytes, PJ_PANEL_BYTES, PJ_PANEL_BYTES + b_stage_bytes, full, empty, 0u, abort_flag,
                           [&](uint32_t a, const CUtensorMap*& mx, const CUtensorMap*& mu, int& m0, int& n0) {
                             const int it = it0 + (int)a * itstep, rem = it % per_tile;
                             const int side = side0 + rem / n_slabs;
                             mx = side ? &map_xv : &map_xk;
                             mu = side ? &map_uv : &map_uk;
                             m0 = (it / per_tile) * TILE;
                             n0 = (rem % n_slabs) * NS;
                           });
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (elect_one())
      ring_gemm_issue<1>(n_acc, KP, PJ_STAGES, sA, stage_bytes, PJ_PANEL_BYTES, idesc_f16(bf16 ? 1 : 0, 128, NS), tmem_base, full, empty,
                         acc_full, acc_empty, abort_flag);
    __syncwarp();
  } else {
    // ------------------------------------------------------------- epilogue
    const int ew = warp - 2;                                   // 0..7
    const int quarter = warp & 3, chalf = ew >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const bool lead_warp = (ew & 3) == 0;                      // one elected lane of this warp issues this half's stores
    unsigned char* my_panel = out_stage + chalf * PJ_PANEL_BYTES;
    const uint32_t my_panel_addr = smem_addr(my_panel);
    const int bar_id = 1 + chalf;
    const int panels = NS / 128;                               // 64-column panels per half slab
    uint32_t ac = 0;
    for (int it = it0; it < n_items; it += itstep, ++ac) {
      const int rem = it % per_tile, m0 = (it / per_tile) * TILE;
      const int side = side0 + rem / n_slabs, ns = rem % n_slabs;
      const CUtensorMap* omap = side ? &map_ov : &map_ok;
      const uint32_t buf = ac & 1u;
      const bool got = mbar_wait(acc_full + 8 * buf, (ac >> 1) & 1u, abort_flag);
      if (!named_bar_and(bar_id, 128, got)) break;             // the four warps of a half leave together
      fence_after_sync();
      for (int pn = 0; pn < panels; ++pn) {
        const int col = chalf * (NS / 2) + pn * 64;            // first column of the panel inside the slab
        float a[32], b[32];
        tmem_ld32(lane_addr + buf * 256 + col, reinterpret_cast<uint32_t*>(a));
        tmem_ld32(lane_addr + buf * 256 + col + 32, reinterpret_cast<uint32_t*>(b));
        tmem_ld_wait();
        if (pn == panels - 1) {                                // last read of this accumulator
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty + 8 * buf);
        }
        uint32_t pk[32];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          pk[u] = bf16 ? pack_bf16x2_rn(a[2 * u], a[2 * u + 1]) : pack_f16x2_rn(a[2 * u], a[2 * u + 1]);
          pk[16 + u] = bf16 ? pack_bf16x2_rn(b[2 * u], b[2 * u + 1]) : pack_f16x2_rn(b[2 * u], b[2 * u + 1]);
        }
        if (lead_warp && elect_one()) bulk_wait_read_all();                      // the previous store has left the staging panel
        named_bar_sync(bar_id, 128);
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8)                         // 16-byte chunk c8 of the row sits at chunk c8 ^ (row % 8)
          *reinterpret_cast<uint4*>(my_panel + row * 128 + ((c8 ^ (row & 7)) << 4)) =
              make_uint4(pk[4 * c8], pk[4 * c8 + 1], pk[4 * c8 + 2], pk[4 * c8 + 3]);
        fence_proxy_async_smem();
        named_bar_sync(bar_id, 128);
        if (lead_warp && elect_one()) {
          tma_store_2d(omap, my_panel_addr, ns * NS + col, m0);
          bulk_commit();
        }
      }
    }
    if (lead_warp && elect_one()) bulk_wait_all();
  }

  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, PJ_TMEM_COLS);
  if (tid == 0 && *abort_flag) atomicCAS(status, 0, TWKV_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// The same product on CTA pairs (cta_group::2): two CTAs of a cluster, on neighbouring SMs, work on one
// [256 x 256] item.  Each loads its own 128 token rows and its own 128 of the slab's 256 rows of U^T, one
// tcgen05.mma of the even CTA drives both tensor cores (M = 256 over the pair, each CTA's accumulator in
// its own TMEM), and each SM reads only half of the B operand from its shared memory: per SM, operand
// traffic from L2 and shared-memory reads both drop from 96 to 64 bytes per tensor-core cycle, which is
// what bounded the single-CTA kernel.  Protocol:
//   full[stage]      lives in the even CTA; both CTAs' copies complete on it (the odd CTA addresses it through
//                    the cluster window), the even CTA's producer lanes post the expected bytes of both
//   empty[stage], acc_full[buf]   one in each CTA, signalled together by a multicast tcgen05.commit
//   acc_empty[buf]   lives in the even CTA; 16 arrivals (8 epilogue warps of each CTA, the odd CTA's remote)
// The cluster barrier brackets the kernel: nobody signals a barrier before it is initialised, nobody leaves
// (and no TMEM is freed) while the partner can still read its shared memory or write its barriers.
constexpr int PJ2_STAGES = 6;
constexpr uint32_t PJ2_STAGE_BYTES = 2 * PJ_PANEL_BYTES;         // [X panel | half of the U^T panel]

__global__ void __launch_bounds__(PJ_THREADS, 1)
project_tc2_kernel(const __grid_constant__ CUtensorMap map_xk, const __grid_constant__ CUtensorMap map_xv,
                   const __grid_constant__ CUtensorMap map_uk, const __grid_constant__ CUtensorMap map_uv,
                   const __grid_constant__ CUtensorMap map_ok, const __grid_constant__ CUtensorMap map_ov,
                   int n_tok, int d, int bf16, int side0, int n_sides, int* status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t crank = cluster_cta_rank();                   // 0 = even CTA: issues the MMAs, owns full / acc_empty
  const int KP = d / PANEL;
  const int n_slabs = d / 256;
  const uint32_t sA = smem_addr(smem_raw);
  const bool misaligned = (sA & 1023u) != 0;
  unsigned char* out_stage = smem_raw + PJ2_STAGES * PJ2_STAGE_BYTES;
  unsigned char* tail = out_stage + 2 * PJ_PANEL_BYTES;
  const uint32_t bars = smem_addr(tail);
  const uint32_t full = bars, empty = full + 8 * PJ2_STAGES, acc_full = empty + 8 * PJ2_STAGES, acc_empty = acc_full + 16;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (2 * PJ2_STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  if (tid == 0) {
    for (int i = 0; i < PJ2_STAGES; ++i) { mbar_init(full + 8 * i, 1); mbar_init(empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 2 * (PJ_EPI / 32)); }
    *abort_flag = misaligned ? 1 : 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc_pair(smem_addr(s_tmem_base), PJ_TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                          // both CTAs' barriers and TMEM are ready
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // item -> (pair of token tiles, side, slab): slab fastest, then side; one item per cluster at a time
  const int per_tile = n_sides * n_slabs;
  const int n_items = per_tile * ((n_tok + 2 * TILE - 1) / (2 * TILE));
  const int it0 = blockIdx.x >> 1, itstep = gridDim.x >> 1;
  const uint32_t n_acc = it0 < n_items ? (uint32_t)((n_items - it0 + itstep - 1) / itstep) : 0u;      // one accumulator per item

  if (misaligned) {
    // nothing was started; fall through to the common exit
  } else if (warp == 0) {
    // ------------------------------------------------------------- TMA producer (both CTAs; one elected thread, ring order)
    if (elect_one()) {
      tma_prefetch_desc(&map_uk); tma_prefetch_desc(&map_uv);
      tma_prefetch_desc(&map_xk); tma_prefetch_desc(&map_xv);
      ring_gemm_produce<2>(n_acc, KP, PJ2_STAGES, sA, PJ2_STAGE_BYTES, PJ_PANEL_BYTES, 4 * PJ_PANEL_BYTES, full, empty, crank, abort_flag,
                           [&](uint32_t a, const CUtensorMap*& mx, const CUtensorMap*& mu, int& m0, int& n0) {
                             const int it = it0 + (int)a * itstep, rem = it % per_tile;
                             const int side = side0 + rem / n_slabs;
                             mx = side ? &map_xv : &map_xk;
                             mu = side ? &map_uv : &map_uk;
                             m0 = (it / per_tile) * (2 * TILE) + (int)crank * TILE;
                             n0 = (rem % n_slabs) * 256 + (int)crank * TILE;
                           });
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (even CTA only)
    if (crank == 0 && elect_one())
      ring_gemm_issue<2>(n_acc, KP, PJ2_STAGES, sA, PJ2_STAGE_BYTES, PJ_PANEL_BYTES, idesc_f16(bf16 ? 1 : 0, 256, 256), tmem_base, full, empty,
                         acc_full, acc_empty, abort_flag);
    __syncwarp();
  } else {
    // ------------------------------------------------------------- epilogue (both CTAs, own 128 rows)
    const int ew = warp - 2;
    const int quarter = warp & 3, chalf = ew >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const bool lead_warp = (ew & 3) == 0;                      // one elected lane of this warp issues this half's stores
    unsigned char* my_panel = out_stage + chalf * PJ_PANEL_BYTES;
    const uint32_t my_panel_addr = smem_addr(my_panel);
    const int bar_id = 1 + chalf;
    const uint32_t acc_empty_even = cluster_map(acc_empty, 0);
    uint32_t ac = 0;
    for (int it = it0; it < n_items; it += itstep, ++ac) {
      const int rem = it % per_tile, m0 = (it / per_tile) * (2 * TILE) + (int)crank * TILE;
      const int side = side0 + rem / n_slabs, ns = rem % n_slabs;
      const CUtensorMap* omap = side ? &map_ov : &map_ok;
      const uint32_t buf = ac & 1u;
      const bool got = mbar_wait(acc_full + 8 * buf, (ac >> 1) & 1u, abort_flag);
      if (!named_bar_and(bar_id, 128, got)) break;
      fence_after_sync();
      for (int pn = 0; pn < 2; ++pn) {
        const int col = chalf * 128 + pn * 64;
        float a[32], b[32];
        tmem_ld32(lane_addr + buf * 256 + col, reinterpret_cast<uint32_t*>(a));
        tmem_ld32(lane_addr + buf * 256 + col + 32, reinterpret_cast<uint32_t*>(b));
        tmem_ld_wait();
        if (pn == 1) {                                         // last read of this accumulator
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_even + 8 * buf);
        }
        uint32_t pk[32];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          pk[u] = bf16 ? pack_bf16x2_rn(a[2 * u], a[2 * u + 1]) : pack_f16x2_rn(a[2 * u], a[2 * u + 1]);
          pk[16 + u] = bf16 ? pack_bf16x2_rn(b[2 * u], b[2 * u + 1]) : pack_f16x2_rn(b[2 * u], b[2 * u + 1]);
        }
        if (lead_warp && elect_one()) bulk_wait_read_all();
        named_bar_sync(bar_id, 128);
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8)
          *reinterpret_cast<uint4*>(my_panel + row * 128 + ((c8 ^ (row & 7)) << 4)) =
              make_uint4(pk[4 * c8], pk[4 * c8 + 1], pk[4 * c8 + 2], pk[4 * c8 + 3]);
        fence_proxy_async_smem();
        named_bar_sync(bar_id, 128);
        if (lead_warp && m0 < n_tok && elect_one()) {                            // the pair's second tile may lie past the last token
          tma_store_2d(omap, my_panel_addr, ns * 256 + col, m0);
          bulk_commit();
        }
      }
    }
    if (lead_warp && elect_one()) bulk_wait_all();
  }

  fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                          // the partner is done with this CTA's memory as well
  fence_after_sync();
  if (warp == 1) tmem_dealloc_pair(tmem_base, PJ_TMEM_COLS);
  if (tid == 0 && *abort_flag) atomicCAS(status, 0, misaligned ? TWKV_ERR_DEVICE_CHECK : TWKV_ERR_TIMEOUT);
}

static void project_pair_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, size_t smem, cudaStream_t st) {
  *cfg = cudaLaunchConfig_t{};
  cfg->blockDim = dim3(PJ_THREADS);
  cfg->dynamicSmemBytes = smem;
  cfg->stream = st;
  attr->id = cudaLaunchAttributeClusterDimension;
  attr->val.clusterDim.x = 2; attr->val.clusterDim.y = 1; attr->val.clusterDim.z = 1;
  cfg->attrs = attr;
  cfg->numAttrs = 1;
}
constexpr size_t PJ2_SMEM = (size_t)PJ2_STAGES * PJ2_STAGE_BYTES + 2 * PJ_PANEL_BYTES + 8 * (2 * PJ2_STAGES + 4) + 16;

// CTA pairs of project_tc2_kernel that can be resident at once on the current device (0: the pair kernel cannot run).
static int project_tc_query_pairs(int sm_count) {
  if (cudaFuncSetAttribute(project_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PJ2_SMEM) != cudaSuccess) { cudaGetLastError(); return 0; }
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr;
  project_pair_config(&cfg, &attr, PJ2_SMEM, nullptr);
  cfg.gridDim = dim3(sm_count & ~1);
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, project_tc2_kernel, &cfg) != cudaSuccess || n < 1) { cudaGetLastError(); n = 0; }
  return n;
}
int project_tc_max_pairs(int sm_count) {
  static const int cached = project_tc_query_pairs(sm_count);  // queried once per process (thread-safe initialisation)
  return cached;
}

cudaError_t launch_project_tc(const ProjectMaps& maps, int n_tok, int d, int bf16, int side0, int n_sides, int* status,
                              int sm_count, bool pairs, cudaStream_t st) {
  if (n_tok <= 0 || n_sides <= 0) return cudaSuccess;
  if (pairs) {
    // maps.uk / maps.uv must have 128-row boxes here (each CTA loads half of a 256-row slab)
    const int max_clusters = project_tc_max_pairs(sm_count);
    if (max_clusters < 1) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(project_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PJ2_SMEM);
    if (e != cudaSuccess) return e;
    const long long n_items = (long long)n_sides * (d / 256) * ((n_tok + 2 * TILE - 1) / (2 * TILE));
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    project_pair_config(&cfg, &attr, PJ2_SMEM, st);
    cfg.gridDim = dim3(2 * (n_items < max_clusters ? (int)n_items : max_clusters));
    e = cudaLaunchKernelEx(&cfg, project_tc2_kernel, maps.xk, maps.xv, maps.uk, maps.uv, maps.ok, maps.ov, n_tok, d, bf16, side0, n_sides, status);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  const int NS = (d % 256 == 0) ? 256 : 128;
  const size_t smem = (size_t)PJ_STAGES * (PJ_PANEL_BYTES + (size_t)NS * 128) + 2 * PJ_PANEL_BYTES + 8 * (2 * PJ_STAGES + 4) + 16;
  cudaError_t e = cudaFuncSetAttribute(project_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long n_items = (long long)n_sides * (d / NS) * ((n_tok + TILE - 1) / TILE);
  const int grid = n_items < sm_count ? (int)n_items : sm_count;
  project_tc_kernel<<<grid, PJ_THREADS, smem, st>>>(maps.xk, maps.xv, maps.uk, maps.uv, maps.ok, maps.ov, n_tok, d, bf16, side0, n_sides, status);
  count_launch();
  return cudaGetLastError();
}

}  // namespace twkv
