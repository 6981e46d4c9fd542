// Gate of the compress step on the 5th-generation tensor cores, logits and rank in one kernel.
//
// Per work item (128 tokens, one side K or V):
//   Z = X~[128 x d] . W[d x d] + b                                             (Eq. 5, the argument of the softmax)
//   p = softmax(Z), c_n = sum_{j<=n} p_j, r = d - #{n : c_n <= tau}            (Eq. 5, Eq. 6, Eq. 8)
// The logits are produced NS columns at a time (NS = 256, or 128 when d is not a multiple of 256) by
// tcgen05.mma chains (M = 128, N = NS, K = 16 per instruction) into two alternating TMEM
// accumulators.  Operands stream through a ring of stages, each one [128 x 64] panel of the token
// tile and one [NS x 64] panel of W (pre-transposed, so it is the K-major B operand), both by TMA with
// the 128-byte swizzle; a token tile of d = 1024 is 256 KB and cannot stay resident, it is re-read
// from L2 once per slab.  CTAs walk the slabs in rotated order so that they do not all ask L2 for
// the same panel of W at the same time.
// Epilogue warps (thread = one token row x half a slab) add the bias, reduce every block of 32 logits
// to (maximum, sum of exp(z - maximum)) in shared memory, and spill the logits to a 128 x d fp32
// staging area owned by the CTA.  Once the item's last slab is out, one thread per row combines the
// block summaries into the softmax denominator, finds the block in which the cumulative sum crosses
// tau and finishes the count inside that block from its 32 staged logits: only 128 bytes per row are
// read back, and the tensor cores already work on the next item meanwhile.
//
// Warp roles (320 threads, one persistent CTA per SM):
//   warp 0      TMA producer: lanes 0-3 the W^T panel of ring stage L, lanes 4-7 the X~ panel of stage L - 4
//               (copies issued by one thread complete one after the other, so every stage has its own two lanes)
//   warp 1      MMA issuer (one elected lane; owns the TMEM allocation)
//   warps 2-9   epilogue and rank
// All waits are bounded (tc_util.cuh); a wait that runs out ends the kernel with TWKV_ERR_TIMEOUT.
#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {
using namespace tc;

constexpr int GT_THREADS = 320;
constexpr int GT_EPI = 256;
constexpr int GT_STAGES = 4;
constexpr uint32_t GT_TMEM_COLS = 512;
constexpr uint32_t GT_PANEL_BYTES = 16384;
constexpr int GT_BLK_STRIDE = 33;                              // row stride of the block summaries (32 blocks + 1 against bank conflicts)

__global__ void __launch_bounds__(GT_THREADS, 1)
gate_tc_kernel(const __grid_constant__ CUtensorMap map_xk, const __grid_constant__ CUtensorMap map_xv,
               const __grid_constant__ CUtensorMap map_wk, const __grid_constant__ CUtensorMap map_wv,
               const float* __restrict__ bias_k, const float* __restrict__ bias_v, int n_tok, int d, int bf16, float tau,
               float* __restrict__ stage_all, unsigned short* __restrict__ levels, int* status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int KP = d / PANEL;                                   // K panels of the token tile
  const int NS = (d % 256 == 0) ? 256 : 128;                  // logits per slab
  const int n_slabs = d / NS;
  const uint32_t b_stage_bytes = (uint32_t)NS * 128u;
  const uint32_t sA = smem_addr(smem_raw);
  if (sA & 1023u) {
    if (tid == 0) atomicCAS(status, 0, TWKV_ERR_DEVICE_CHECK);
    return;
  }
  const uint32_t stage_bytes = GT_PANEL_BYTES + b_stage_bytes;           // [X~ panel | W^T panel]
  float2* sBlk = reinterpret_cast<float2*>(smem_raw + GT_STAGES * stage_bytes);   // [128 rows][33]: (max, sum of exp) per block of 32 logits
  unsigned char* tail = smem_raw + GT_STAGES * stage_bytes + TILE * GT_BLK_STRIDE * sizeof(float2);
  const uint32_t bars = smem_addr(tail);
  // barrier map (8 bytes each)
  const uint32_t full = bars, empty = full + 8 * GT_STAGES, acc_full = empty + 8 * GT_STAGES, acc_empty = acc_full + 16;
  const uint32_t epi_bar = acc_empty + 16;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (2 * GT_STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  if (tid == 0) {
    for (int i = 0; i < GT_STAGES; ++i) { mbar_init(full + 8 * i, 2); mbar_init(empty + 8 * i, 1); }   // two copies fill a stage
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, GT_EPI / 32); }
    mbar_init(epi_bar, GT_EPI);
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(smem_addr(s_tmem_base), GT_TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // work items: (token tile, side), the two sides of a tile next to each other
  const int n_items = 2 * ((n_tok + TILE - 1) / TILE);
  const int it0 = blockIdx.x, itstep = gridDim.x;

  const int ns_rot = blockIdx.x % n_slabs;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane < 2 * GT_STAGES) {
      const bool is_x = lane >= GT_STAGES;
      const uint32_t my = is_x ? lane - GT_STAGES : lane;      // the ring stage this lane serves
      if (lane == 0) { tma_prefetch_desc(&map_wk); tma_prefetch_desc(&map_wv); }
      if (lane == GT_STAGES) { tma_prefetch_desc(&map_xk); tma_prefetch_desc(&map_xv); }
      bool ok = true;
      uint32_t st = 0, ph = 0;
      for (int it = it0; it < n_items && ok; it += itstep) {
        const int m0 = (it >> 1) * TILE;
        const CUtensorMap* map = is_x ? ((it & 1) ? &map_xv : &map_xk) : ((it & 1) ? &map_wv : &map_wk);
        for (int sl = 0; sl < n_slabs && ok; ++sl) {
          const int ns = sl + ns_rot < n_slabs ? sl + ns_rot : sl + ns_rot - n_slabs;
          for (int p = 0; p < KP; ++p) {
            const uint32_t cst = st, cph = ph;
            if (++st == GT_STAGES) { st = 0; ph ^= 1u; }
            if (cst != my) continue;
            if (!(ok = mbar_wait(empty + 8 * cst, cph ^ 1u, abort_flag))) break;
            if (is_x) {
              mbar_expect_tx(full + 8 * cst, GT_PANEL_BYTES);
              tma_load_2d(sA + cst * stage_bytes, map, full + 8 * cst, p * PANEL, m0);
            } else {
              mbar_expect_tx(full + 8 * cst, b_stage_bytes);
              tma_load_2d(sA + cst * stage_bytes + GT_PANEL_BYTES, map, full + 8 * cst, p * PANEL, ns * NS);
            }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (elect_one()) {
      const uint32_t idesc = idesc_f16(bf16 ? 1 : 0, 128, NS);
      const uint64_t adesc0 = kmajor_sw128_desc(sA), bdesc0 = kmajor_sw128_desc(sA + GT_PANEL_BYTES);
      bool ok = true;
      uint32_t st = 0, ph = 0, ac = 0;
      for (int it = it0; it < n_items && ok; it += itstep) {
        for (int sl = 0; sl < n_slabs && ok; ++sl, ++ac) {
          const uint32_t buf = ac & 1u;
          if (!(ok = mbar_wait(acc_empty + 8 * buf, ((ac >> 1) & 1u) ^ 1u, abort_flag))) break;
          const uint32_t dcol = tmem_base + buf * 256;
          for (int p = 0; p < KP; ++p) {
            const uint32_t cst = st, cph = ph;
            if (++st == GT_STAGES) { st = 0; ph ^= 1u; }
            if (!(ok = mbar_wait(full + 8 * cst, cph, abort_flag))) break;
            fence_after_sync();
            const uint64_t adesc = adesc0 + (uint64_t)(cst * (stage_bytes >> 4));
            const uint64_t bdesc = bdesc0 + (uint64_t)(cst * (stage_bytes >> 4));
            mma_f16_ss(dcol, adesc, bdesc, idesc, p > 0 ? 1u : 0u);
#pragma unroll
            for (int ks = 1; ks < 4; ++ks) mma_f16_ss(dcol, adesc + 2 * ks, bdesc + 2 * ks, idesc, 1u);
            mma_commit(empty + 8 * cst);
          }
          if (!ok) break;
          mma_commit(acc_full + 8 * buf);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------- epilogue + rank
    const int ew = warp - 2;                                   // 0..7
    const int quarter = warp & 3, chalf = ew >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    // this CTA's staging area, layout [d / 4][128 rows][4 floats]: the 32 rows of a warp store 512 contiguous bytes per instruction
    float* stage = stage_all + (size_t)blockIdx.x * TILE * d;
    const int cols_per_thread = NS / 2;                        // each row of a slab is split between two threads
    uint32_t ac = 0, epar = 0;
    bool ok = true;
    auto epi_sync = [&]() {
      mbar_arrive(epi_bar);
      const bool r = __all_sync(0xffffffffu, mbar_wait(epi_bar, epar, abort_flag));
      epar ^= 1u;
      return r;
    };
    for (int it = it0; it < n_items && ok; it += itstep) {
      const int m0 = (it >> 1) * TILE, side = it & 1;
      const float* bias = side ? bias_v : bias_k;
      for (int sl = 0; sl < n_slabs && ok; ++sl, ++ac) {
        const int ns = sl + ns_rot < n_slabs ? sl + ns_rot : sl + ns_rot - n_slabs;
        const uint32_t buf = ac & 1u;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(acc_full + 8 * buf, (ac >> 1) & 1u, abort_flag)))) break;
        fence_after_sync();
        const int col0 = ns * NS + chalf * cols_per_thread;
        float* dst = stage + (size_t)(col0 >> 2) * (TILE * 4) + row * 4;
        for (int c = 0; c < cols_per_thread; c += 32) {
          float z[32];
          tmem_ld32(lane_addr + buf * 256 + chalf * cols_per_thread + c, reinterpret_cast<uint32_t*>(z));
          tmem_ld_wait();
          if (c + 32 >= cols_per_thread) {                                  // last read of this accumulator
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty + 8 * buf);
          }
          float bm = -INFINITY;
#pragma unroll
          for (int u = 0; u < 32; u += 4) {
            if (bias) {
              const float4 bb = __ldg(reinterpret_cast<const float4*>(bias + col0 + c + u));
              z[u] += bb.x; z[u + 1] += bb.y; z[u + 2] += bb.z; z[u + 3] += bb.w;
            }
            __stcg(reinterpret_cast<float4*>(dst + (size_t)((c + u) >> 2) * (TILE * 4)), make_float4(z[u], z[u + 1], z[u + 2], z[u + 3]));
            bm = fmaxf(bm, fmaxf(fmaxf(z[u], z[u + 1]), fmaxf(z[u + 2], z[u + 3])));
          }
          // block of 32 logits: its maximum and the sum of exp(z - maximum)
          float bs = 0.f;
#pragma unroll
          for (int u = 0; u < 32; ++u) bs += __expf(z[u] - bm);
          sBlk[row * GT_BLK_STRIDE + ((col0 + c) >> 5)] = make_float2(bm, bs);
        }
      }
      if (!ok) break;
      if (!(ok = epi_sync())) break;                           // every block summary and every staged logit of the item is out
      // rank (Eq. 6, Eq. 8), one thread per row: combine the block summaries into the row total S_d, walk the blocks to
      // the one where the running sum crosses tau * S_d, and finish inside that block from its 32 staged logits
      if (ew < 4) {
        const int rr = ew * 32 + lane;
        if (m0 + rr < n_tok) {
          const float2* blk = sBlk + rr * GT_BLK_STRIDE;
          const int nblk = d >> 5;
          float M = -INFINITY;
          for (int b = 0; b < nblk; ++b) M = fmaxf(M, blk[b].x);
          float total = 0.f;
          for (int b = 0; b < nblk; ++b) total += blk[b].y * __expf(blk[b].x - M);
          const float thr = tau * total;                        // c_n <= tau  <=>  S_n <= tau * S_d
          float run = 0.f, base = 0.f;
          int bstar = -1;
          for (int b = 0; b < nblk; ++b) {
            const float t = blk[b].y * __expf(blk[b].x - M);
            if (bstar < 0 && run + t > thr) { bstar = b; base = run; }
            run += t;
          }
          int below = d;                                        // NaN logits: nothing crosses, r clamps to 1
          if (bstar >= 0) {
            const float* zb = stage + (size_t)(bstar * 8) * (TILE * 4) + rr * 4;
            float sn = base;
            int cnt = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float4 t = __ldcg(reinterpret_cast<const float4*>(zb + (size_t)u * (TILE * 4)));
              sn += __expf(t.x - M); cnt += sn <= thr ? 1 : 0;
              sn += __expf(t.y - M); cnt += sn <= thr ? 1 : 0;
              sn += __expf(t.z - M); cnt += sn <= thr ? 1 : 0;
              sn += __expf(t.w - M); cnt += sn <= thr ? 1 : 0;
            }
            below = bstar * 32 + cnt;
          }
          int r = d - below;
          if (r < 1) r = 1;
          levels[(size_t)(m0 + rr) * 2 + side] = (unsigned short)r;
        }
      }
      if (!(ok = epi_sync())) break;                           // the staging area may be overwritten by the next item
    }
  }

  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, GT_TMEM_COLS);
  if (tid == 0 && *abort_flag) atomicCAS(status, 0, TWKV_ERR_TIMEOUT);
}

size_t gate_tc_stage_bytes(int n_cta, int d) { return (size_t)n_cta * TILE * d * sizeof(float); }

cudaError_t launch_gate_ranks_tc(const DevView& v, const GateMaps& maps, const LayerParams& lp, int n_tok, unsigned short* levels,
                                 int sm_count, cudaStream_t st) {
  if (n_tok <= 0) return cudaSuccess;
  const int d = v.d_kv;
  const int NS = (d % 256 == 0) ? 256 : 128;
  const size_t smem = (size_t)GT_STAGES * (GT_PANEL_BYTES + (size_t)NS * 128) + TILE * GT_BLK_STRIDE * sizeof(float2) + 8 * (2 * GT_STAGES + 5) + 16;
  cudaError_t e = cudaFuncSetAttribute(gate_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int n_items = 2 * ((n_tok + TILE - 1) / TILE);
  const int grid = n_items < sm_count ? n_items : sm_count;
  {
    ProfScope ps(TWKV_K_GATE_GEMM, st);
    gate_tc_kernel<<<grid, GT_THREADS, smem, st>>>(maps.xk, maps.xv, maps.wk, maps.wv, lp.b_k, lp.b_v, n_tok, d,
                                                   v.dtype == TWKV_BF16 ? 1 : 0, v.tau, v.gate_scratch, levels, v.status);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace twkv
