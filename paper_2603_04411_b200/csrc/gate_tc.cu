// Gate of the compress step on the 5th-generation tensor cores, logits and rank in one kernel.
//
// Per work item (128 tokens, one side K or V):
//   Z = X~[128 x d] . W[d x d] + b                                             (Eq. 5, the argument of the softmax)
//   p = softmax(Z), c_n = sum_{j<=n} p_j, r = d - #{n : c_n <= tau}            (Eq. 5, Eq. 6, Eq. 8)
// The logits are produced NS columns at a time (NS = 256, or 128 when d is not a multiple of 256) by
// tcgen05.mma chains (K = 16 per instruction) into two alternating TMEM accumulators.  Operands stream
// through a ring of stages, each one [128 x 64] panel of the token tile and one panel of W (pre-transposed,
// so it is the K-major B operand), both by TMA with the 128-byte swizzle; a token tile of d = 1024 is 256 KB
// and cannot stay resident, it is re-read from L2 once per slab.  CTAs walk the slabs in rotated order so
// that they do not all ask L2 for the same panel of W at the same time.
// Epilogue warps (thread = one token row x half a slab) add the bias, reduce every block of 32 logits to
// (maximum, sum of exp(z - maximum)) in shared memory, and stage the 32 terms exp(z - maximum) as f16 in a
// 128 x d block of global memory owned by the CTA, written and read with an L2 "evict last" policy so that
// it stays in L2 (in fp32 and without the policy most of it was written back to DRAM behind the streamed
// states, and the kernel took 1.4x as long).  Once the item's last slab is out, two threads per row combine
// the block summaries into the softmax denominator, find the block in which the cumulative sum crosses tau
// and finish the count inside that block from its 32 staged terms: 64 bytes per row are read back, and the
// tensor cores already work on the next item meanwhile.
//
// Two kernels share that epilogue: gate_tc2_kernel on CTA pairs (d a multiple of 256, the usual case) and
// gate_tc_kernel on single CTAs.  Warp roles (320 threads, one persistent CTA per SM):
//   warp 0      TMA producer: one lane per copy and ring stage (copies issued by one thread complete one after
//               the other, so every stage has its own two lanes)
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

// L2 eviction policy "keep": the logits staging block is rewritten for every item and only read back in the
// same item, so it should stay in L2 instead of being written back to DRAM behind the streamed states.
__device__ __forceinline__ uint64_t l2_keep_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_keep_v4(void* ptr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;"
               ::"l"(ptr), "r"(a), "r"(b), "r"(c), "r"(d), "l"(policy) : "memory");
}
__device__ __forceinline__ uint4 ld_keep_v4(const void* ptr, uint64_t policy) {
  uint4 v;
  asm volatile("ld.global.cg.L2::cache_hint.v4.b32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr), "l"(policy) : "memory");
  return v;
}
__device__ __forceinline__ float2 unpack_f16x2(uint32_t v) {
  float2 r;
  asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.f32.f16 %0, lo;\n\tcvt.f32.f16 %1, hi;\n\t}" : "=f"(r.x), "=f"(r.y) : "r"(v));
  return r;
}

// One row decided again in fp32 by a whole warp (Eq. 5, 6, 8 for the 32 logits of the block in which the cumulative
// sum crosses tau): every logit is a dot product over d spread across the lanes (coalesced reads of the transposed
// weights, butterfly sum), the terms exp(z - M) continue the cumulative sum from `base`, the block summaries before
// the crossing block having been taken in fp32 already.
__device__ __forceinline__ void gate_redo_row(const GateRaw& raw, int bf16, int d, const float* __restrict__ bias_k,
                                              const float* __restrict__ bias_v, int side, int row, int b_s, float base, float thr,
                                              float M, unsigned short* __restrict__ levels, int lane) {
  const int n16 = d >> 3;                                      // 16-byte pieces per row; lane takes pieces lane, lane + 32, ...
  auto widen = [&](const uint4 q, float* f) {
    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (bf16) { f[2 * k] = __uint_as_float(w4[k] << 16); f[2 * k + 1] = __uint_as_float(w4[k] & 0xffff0000u); }
      else { const float2 t = unpack_f16x2(w4[k]); f[2 * k] = t.x; f[2 * k + 1] = t.y; }
    }
  };
  float xf[32];
  {
    const uint4* xr = reinterpret_cast<const uint4*>((side ? raw.xv : raw.xk) + (size_t)row * d);
#pragma unroll
    for (int k = 0; k < 4; ++k) widen(lane + 32 * k < n16 ? __ldg(xr + lane + 32 * k) : make_uint4(0u, 0u, 0u, 0u), xf + 8 * k);
  }
  const unsigned short* wbase = (side ? raw.wvT : raw.wkT) + (size_t)(b_s * 32) * d;
  float z = 0.f;
#pragma unroll 1
  for (int j0 = 0; j0 < 32; j0 += 4) {
    uint4 wq[4][4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const uint4* wr = reinterpret_cast<const uint4*>(wbase + (size_t)(j0 + jj) * d);
#pragma unroll
      for (int k = 0; k < 4; ++k) wq[jj][k] = lane + 32 * k < n16 ? __ldg(wr + lane + 32 * k) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      float acc = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float wf[8];
        widen(wq[jj][k], wf);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fmaf(xf[8 * k + e], wf[e], acc);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (lane == j0 + jj) z = acc;
    }
  }
  const float* bias = side ? bias_v : bias_k;
  if (bias) z += __ldg(bias + b_s * 32 + lane);
  float incl = __expf(z - M);
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  const int cnt = __popc(__ballot_sync(0xffffffffu, base + incl <= thr));
  if (lane == 0) {
    int r = d - (b_s * 32 + cnt);
    if (r < 1) r = 1;
    levels[(size_t)row * 2 + side] = (unsigned short)r;
  }
}

// The rows the fused kernel could not decide from its f16-staged terms, one warp per row.  The list's counter is
// cleared by the last CTA to finish, so the next launch of the fused kernel starts from an empty list.
constexpr int GT_FIX_CAP = 1 << 18;                            // list entries; rows beyond are decided inside the fused kernel
constexpr int GT_FIX_THREADS = 128;
__global__ void __launch_bounds__(GT_FIX_THREADS)
gate_fixup_kernel(const GateRaw raw, int bf16, int d, const float* __restrict__ bias_k, const float* __restrict__ bias_v,
                  const int4* __restrict__ list, int* counters, unsigned short* __restrict__ levels) {
  const int lane = threadIdx.x & 31;
  const int n = min(counters[0], GT_FIX_CAP);
  for (int i = (blockIdx.x * GT_FIX_THREADS + threadIdx.x) >> 5; i < n; i += (gridDim.x * GT_FIX_THREADS) >> 5) {
    const int4 e0 = list[2 * i], e1 = list[2 * i + 1];
    gate_redo_row(raw, bf16, d, bias_k, bias_v, e0.y & 1, e0.x, e0.y >> 1, __int_as_float(e0.z), __int_as_float(e0.w),
                  __int_as_float(e1.x), levels, lane);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&counters[1], 1) == (int)gridDim.x - 1) { counters[0] = 0; counters[1] = 0; __threadfence(); }
  }
}

// Epilogue and rank role of both gate kernels (warps 2-9, 256 threads).
//   Per slab: thread = (token row, half of the slab's columns).  Every block of 32 logits is reduced to
//   (maximum bm, sum of exp(z - bm)) in shared memory, and the 32 terms exp(z - bm), which lie in (0, 1], are
//   staged as f16 in the CTA's staging block, laid out [d / 8][128 rows][8] so that a warp's stores are contiguous.
//   Per item: thread = (token row, half of the row's blocks), the two halves of a row in neighbouring lanes.
//   Both combine the block summaries into the softmax denominator S_d, the half that holds the block in which
//   the running sum crosses tau * S_d finishes inside it from the block's 32 staged terms (64 bytes per row).
//   The f16 rounding of the staged terms moves a cumulative sum by at most 2^-11 of its block's share of S_d,
//   i.e. by less than 0.5 % of tau = 0.1.  A row whose decision is closer than that bound is decided again from
//   fp32 terms (the warp recomputes the crossing block's 32 logits from the 16-bit operands), so the rank this
//   kernel writes has the accuracy of an fp32 evaluation of Eq. 5, 6 and 8, like the small-call path.
// PAIR: the kernel runs on CTA pairs; the accumulator-free barrier lives in the even CTA and rows start at
// the CTA's own half of the 256-token item.
template <bool PAIR>
__device__ __forceinline__ void gate_epilogue_role(uint32_t tmem_base, uint32_t acc_full, uint32_t acc_empty, uint32_t epi_bar,
                                                   float2* sBlk, volatile int* abort_flag, unsigned short* stage,
                                                   const float* __restrict__ bias_k, const float* __restrict__ bias_v,
                                                   unsigned short* __restrict__ levels, int n_tok, int d, int NS, int n_slabs,
                                                   int ns_rot, int it0, int itstep, int n_items, float tau, uint32_t crank,
                                                   const GateRaw raw, int bf16, int* status) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ew = warp - 2;                                   // 0..7
  const int quarter = warp & 3, chalf = ew >> 2;
  const int row = quarter * 32 + lane;
  const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
  const int cols_per_thread = NS / 2;                        // each row of a slab is split between two threads
  const uint32_t acc_empty_owner = PAIR ? cluster_map(acc_empty, 0) : acc_empty;
  const uint64_t keep = l2_keep_policy();
  // rank step mapping: row rr, half hh of its blocks
  const int et = ew * 32 + lane, rr = et >> 1, hh = et & 1;
  uint32_t ac = 0, epar = 0;
  bool ok = true;
  auto epi_sync = [&]() {
    mbar_arrive(epi_bar);
    const bool r = __all_sync(0xffffffffu, mbar_wait(epi_bar, epar, abort_flag));
    epar ^= 1u;
    return r;
  };
  for (int it = it0; it < n_items && ok; it += itstep) {
    const int m0 = PAIR ? (it >> 1) * (2 * TILE) + (int)crank * TILE : (it >> 1) * TILE;
    const int side = it & 1;
    const float* bias = side ? bias_v : bias_k;
    for (int sl = 0; sl < n_slabs && ok; ++sl, ++ac) {
      const int ns = sl + ns_rot < n_slabs ? sl + ns_rot : sl + ns_rot - n_slabs;
      const uint32_t buf = ac & 1u;
      if (!(ok = __all_sync(0xffffffffu, mbar_wait(acc_full + 8 * buf, (ac >> 1) & 1u, abort_flag)))) break;
      fence_after_sync();
      const int col0 = ns * NS + chalf * cols_per_thread;
      unsigned short* dst = stage + ((size_t)(col0 >> 3) * TILE + row) * 8;
      for (int c = 0; c < cols_per_thread; c += 32) {
        float z[32];
        tmem_ld32(lane_addr + buf * 256 + chalf * cols_per_thread + c, reinterpret_cast<uint32_t*>(z));
        tmem_ld_wait();
        if (c + 32 >= cols_per_thread) {                                  // last read of this accumulator
          fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(acc_empty_owner + 8 * buf);
            else mbar_arrive(acc_empty_owner + 8 * buf);
          }
        }
        float bm = -INFINITY;
#pragma unroll
        for (int u = 0; u < 32; u += 4) {
          if (bias) {
            const float4 bb = __ldg(reinterpret_cast<const float4*>(bias + col0 + c + u));
            z[u] += bb.x; z[u + 1] += bb.y; z[u + 2] += bb.z; z[u + 3] += bb.w;
          }
          bm = fmaxf(bm, fmaxf(fmaxf(z[u], z[u + 1]), fmaxf(z[u + 2], z[u + 3])));
        }
        // block of 32 logits: its maximum, the sum of exp(z - maximum), and the 32 terms themselves
        float bs = 0.f;
#pragma unroll
        for (int u = 0; u < 32; ++u) { z[u] = __expf(z[u] - bm); bs += z[u]; }
#pragma unroll
        for (int u = 0; u < 32; u += 8)
          st_keep_v4(dst + (size_t)((c + u) >> 3) * (TILE * 8), pack_f16x2_sat(z[u], z[u + 1]), pack_f16x2_sat(z[u + 2], z[u + 3]),
                     pack_f16x2_sat(z[u + 4], z[u + 5]), pack_f16x2_sat(z[u + 6], z[u + 7]), keep);
        sBlk[row * GT_BLK_STRIDE + ((col0 + c) >> 5)] = make_float2(bm, bs);
      }
    }
    if (!ok) break;
    if (!(ok = epi_sync())) break;                           // every block summary and every staged term of the item is out
    // rank (Eq. 6, Eq. 8): lanes 2k / 2k + 1 take the lower / upper half of row rr's blocks
    {
      const float2* blk = sBlk + rr * GT_BLK_STRIDE;
      const int half = d >> 6, b0 = hh * half;               // d / 32 blocks per row, an even number
      float m = -INFINITY;
      for (int b = b0; b < b0 + half; ++b) m = fmaxf(m, blk[b].x);
      const float M = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
      float s = 0.f;
      for (int b = b0; b < b0 + half; ++b) s += blk[b].y * __expf(blk[b].x - M);
      const float so = __shfl_xor_sync(0xffffffffu, s, 1);
      const float lo = hh ? so : s, hi = hh ? s : so;
      const float thr = tau * (lo + hi);                     // c_n <= tau  <=>  S_n <= tau * S_d
      // a row with a NaN or an infinite logit has no softmax: its rank is a placeholder, the call reports it
      if (hh == 0 && m0 + rr < n_tok && !(thr > 0.f && thr < INFINITY)) atomicCAS(status, 0, TWKV_ERR_DEVICE_CHECK);
      float run = hh ? lo : 0.f, base = 0.f;
      int bstar = -1;
      for (int b = b0; b < b0 + half; ++b) {
        const float t = blk[b].y * __expf(blk[b].x - M);
        if (bstar < 0 && run + t > thr) { bstar = b; base = run; }
        run += t;
      }
      const bool lower_found = __shfl_sync(0xffffffffu, bstar >= 0 ? 1 : 0, lane & ~1) != 0;
      const bool mine = hh ? !lower_found : bstar >= 0;      // the upper half also reports "nothing crossed" (NaN logits: r = 1)
      bool redo = false;                                     // decided closer to tau than the f16 staging can tell
      if (mine && m0 + rr < n_tok) {
        int below = d;
        if (bstar >= 0) {
          const float scale = __expf(blk[bstar].x - M);
          // a staged term is off by at most 2^-11 of itself (round to nearest), or 2^-25 once it is subnormal in f16,
          // so the cumulative sum after k terms is off by at most 2^-11 of the block's partial sum + k 2^-25
          const unsigned short* zb = stage + ((size_t)(bstar * 4) * TILE + rr) * 8;
          float sn = base, part = 0x1p-20f;                  // part: the block's partial sum (+ the subnormal allowance)
          int cnt = 0;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint4 t = ld_keep_v4(zb + (size_t)u * (TILE * 8), keep);
            const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float2 e = unpack_f16x2(w[k]);
              sn += e.x * scale; part += e.x; cnt += sn <= thr ? 1 : 0; redo |= fabsf(sn - thr) <= part * scale * 0x1.2p-11f;
              sn += e.y * scale; part += e.y; cnt += sn <= thr ? 1 : 0; redo |= fabsf(sn - thr) <= part * scale * 0x1.2p-11f;
            }
          }
          below = bstar * 32 + cnt;
        }
        int r = d - below;
        if (r < 1) r = 1;
        if (!redo) levels[(size_t)(m0 + rr) * 2 + side] = (unsigned short)r;
      }
      // Rows flagged above are decided again in fp32 (gate_redo_row) by the small kernel that follows this one; the
      // list holds what it needs.  Should the list ever be full, the warp does the row here instead.
      if (redo) {
        const int slot = atomicAdd(raw.fix_counters, 1);
        if (slot < GT_FIX_CAP) {
          raw.fix_list[2 * slot] = make_int4(m0 + rr, side | (bstar << 1), __float_as_int(base), __float_as_int(thr));
          raw.fix_list[2 * slot + 1] = make_int4(__float_as_int(M), 0, 0, 0);
          redo = false;
        }
      }
      unsigned todo = __ballot_sync(0xffffffffu, redo);
      while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        gate_redo_row(raw, bf16, d, bias_k, bias_v, side, m0 + __shfl_sync(0xffffffffu, rr, src), __shfl_sync(0xffffffffu, bstar, src),
                      __shfl_sync(0xffffffffu, base, src), __shfl_sync(0xffffffffu, thr, src), __shfl_sync(0xffffffffu, M, src),
                      levels, lane);
      }
    }
    if (!(ok = epi_sync())) break;                           // the staging block may be overwritten by the next item
  }
}

__global__ void __launch_bounds__(GT_THREADS, 1)
gate_tc_kernel(const __grid_constant__ CUtensorMap map_xk, const __grid_constant__ CUtensorMap map_xv,
               const __grid_constant__ CUtensorMap map_wk, const __grid_constant__ CUtensorMap map_wv,
               const float* __restrict__ bias_k, const float* __restrict__ bias_v, int n_tok, int d, int bf16, float tau,
               float* __restrict__ stage_all, unsigned short* __restrict__ levels, int* status, const GateRaw raw) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5;
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
    for (int i = 0; i < GT_STAGES; ++i) { mbar_init(full + 8 * i, 1); mbar_init(empty + 8 * i, 1); }   // the producer posts both copies' bytes
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
  // accumulators this CTA produces: its items x the slabs of an item
  const uint32_t n_acc = it0 < n_items ? (uint32_t)((n_items - it0 + itstep - 1) / itstep) * (uint32_t)n_slabs : 0u;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer (one elected thread, ring order)
    if (elect_one()) {
      tma_prefetch_desc(&map_wk); tma_prefetch_desc(&map_wv);
      tma_prefetch_desc(&map_xk); tma_prefetch_desc(&map_xv);
      ring_gemm_produce<1>(n_acc, KP, GT_STAGES, sA, stage_bytes, GT_PANEL_BYTES, GT_PANEL_BYTES + b_stage_bytes, full, empty, 0u, abort_flag,
                           [&](uint32_t a, const CUtensorMap*& mx, const CUtensorMap*& mw, int& m0, int& n0) {
                             const int it = it0 + (int)(a / (uint32_t)n_slabs) * itstep, sl = (int)(a % (uint32_t)n_slabs);
                             const int ns = sl + ns_rot < n_slabs ? sl + ns_rot : sl + ns_rot - n_slabs;
                             mx = (it & 1) ? &map_xv : &map_xk;
                             mw = (it & 1) ? &map_wv : &map_wk;
                             m0 = (it >> 1) * TILE;
                             n0 = ns * NS;
                           });
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (elect_one())
      ring_gemm_issue<1>(n_acc, KP, GT_STAGES, sA, stage_bytes, GT_PANEL_BYTES, idesc_f16(bf16 ? 1 : 0, 128, NS), tmem_base, full, empty,
                         acc_full, acc_empty, abort_flag);
    __syncwarp();
  } else {
    // ------------------------------------------------------------- epilogue + rank
    gate_epilogue_role<false>(tmem_base, acc_full, acc_empty, epi_bar, sBlk, abort_flag,
                              reinterpret_cast<unsigned short*>(stage_all) + (size_t)blockIdx.x * TILE * d, bias_k, bias_v, levels,
                              n_tok, d, NS, n_slabs, ns_rot, it0, itstep, n_items, tau, 0u, raw, bf16, status);
  }

  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, GT_TMEM_COLS);
  if (tid == 0 && *abort_flag) atomicCAS(status, 0, TWKV_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// The same kernel on CTA pairs (cta_group::2), used when d is a multiple of 256: the two CTAs of a cluster take
// 256 consecutive tokens, each loads its own 128 token rows and its own 128 of the slab's 256 rows of W^T, one
// tcgen05.mma of the even CTA drives both tensor cores (M = 256 over the pair, each CTA's accumulator in its own
// TMEM) and each SM reads only half of the B operand from its shared memory.  Per SM the operand traffic from L2
// and the shared-memory reads both drop from 96 to 64 bytes per tensor-core cycle, which is what held the
// single-CTA kernel at about half of the tensor pipe.  Barriers: full[stage] and acc_empty[buf] live in the even
// CTA (the odd CTA's copies complete on them / its epilogue warps arrive on them through the cluster window);
// empty[stage] and acc_full[buf] exist in both and are signalled together by a multicast tcgen05.commit.  The
// epilogue and the rank step are per CTA, unchanged.  The cluster barrier brackets the kernel: nobody signals a
// barrier before it is initialised, and nobody leaves (no TMEM is freed) while its partner can still read its
// shared memory or write its barriers.
constexpr int GT2_STAGES = 6;

__global__ void __launch_bounds__(GT_THREADS, 1)
gate_tc2_kernel(const __grid_constant__ CUtensorMap map_xk, const __grid_constant__ CUtensorMap map_xv,
               const __grid_constant__ CUtensorMap map_wk, const __grid_constant__ CUtensorMap map_wv,
               const float* __restrict__ bias_k, const float* __restrict__ bias_v, int n_tok, int d, int bf16, float tau,
               float* __restrict__ stage_all, unsigned short* __restrict__ levels, int* status, const GateRaw raw) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t crank = cluster_cta_rank();                  // 0 = even CTA: issues the MMAs, owns full / acc_empty
  const int KP = d / PANEL;                                   // K panels of the token tile
  constexpr int NS = 256;                                     // logits per slab (d is a multiple of 256 here)
  const int n_slabs = d / NS;
  const uint32_t sA = smem_addr(smem_raw);
  const bool misaligned = (sA & 1023u) != 0;
  constexpr uint32_t stage_bytes = 2 * GT_PANEL_BYTES;                   // [X~ panel | this CTA's half of the W^T panel]
  float2* sBlk = reinterpret_cast<float2*>(smem_raw + GT2_STAGES * stage_bytes);   // [128 rows][33]: (max, sum of exp) per block of 32 logits
  unsigned char* tail = smem_raw + GT2_STAGES * stage_bytes + TILE * GT_BLK_STRIDE * sizeof(float2);
  const uint32_t bars = smem_addr(tail);
  // barrier map (8 bytes each)
  const uint32_t full = bars, empty = full + 8 * GT2_STAGES, acc_full = empty + 8 * GT2_STAGES, acc_empty = acc_full + 16;
  const uint32_t epi_bar = acc_empty + 16;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (2 * GT2_STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  if (tid == 0) {
    for (int i = 0; i < GT2_STAGES; ++i) { mbar_init(full + 8 * i, 1); mbar_init(empty + 8 * i, 1); }   // even CTA: its producer posts both CTAs' bytes
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 2 * (GT_EPI / 32)); }
    mbar_init(epi_bar, GT_EPI);
    *abort_flag = misaligned ? 1 : 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc_pair(smem_addr(s_tmem_base), GT_TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                         // both CTAs' barriers and TMEM are ready
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // work items: (pair of token tiles, side), the two sides of a pair next to each other; one item per cluster at a time
  const int n_items = 2 * ((n_tok + 2 * TILE - 1) / (2 * TILE));
  const int it0 = blockIdx.x >> 1, itstep = gridDim.x >> 1;

  const int ns_rot = (blockIdx.x >> 1) % n_slabs;
  // accumulators this pair produces: its items x the slabs of an item
  const uint32_t n_acc = it0 < n_items ? (uint32_t)((n_items - it0 + itstep - 1) / itstep) * (uint32_t)n_slabs : 0u;

  if (misaligned) {
    // nothing was started; fall through to the common exit
  } else if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    // One elected thread issues every copy in ring order (stages free up in that order): a copy instruction issued
    // from a lane picked by its index costs that warp hundreds of cycles, and lanes of one warp that wait on different
    // barriers wait one after the other.
    if (elect_one()) {
      tma_prefetch_desc(&map_wk); tma_prefetch_desc(&map_wv);
      tma_prefetch_desc(&map_xk); tma_prefetch_desc(&map_xv);
      ring_gemm_produce<2>(n_acc, KP, GT2_STAGES, sA, stage_bytes, GT_PANEL_BYTES, 4 * GT_PANEL_BYTES, full, empty, crank, abort_flag,
                           [&](uint32_t a, const CUtensorMap*& mx, const CUtensorMap*& mw, int& m0, int& n0) {
                             const int it = it0 + (int)(a / (uint32_t)n_slabs) * itstep, sl = (int)(a % (uint32_t)n_slabs);
                             const int ns = sl + ns_rot < n_slabs ? sl + ns_rot : sl + ns_rot - n_slabs;
                             mx = (it & 1) ? &map_xv : &map_xk;
                             mw = (it & 1) ? &map_wv : &map_wk;
                             m0 = (it >> 1) * (2 * TILE) + (int)crank * TILE;
                             n0 = ns * NS + (int)crank * TILE;
                           });
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (even CTA only)
    if (crank == 0 && elect_one())
      ring_gemm_issue<2>(n_acc, KP, GT2_STAGES, sA, stage_bytes, GT_PANEL_BYTES, idesc_f16(bf16 ? 1 : 0, 256, NS), tmem_base, full, empty,
                         acc_full, acc_empty, abort_flag);
    __syncwarp();
  } else {
    // ------------------------------------------------------------- epilogue + rank
    gate_epilogue_role<true>(tmem_base, acc_full, acc_empty, epi_bar, sBlk, abort_flag,
                              reinterpret_cast<unsigned short*>(stage_all) + (size_t)blockIdx.x * TILE * d, bias_k, bias_v, levels,
                              n_tok, d, NS, n_slabs, ns_rot, it0, itstep, n_items, tau, crank, raw, bf16, status);
  }

  fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                         // the partner is done with this CTA's memory as well
  fence_after_sync();
  if (warp == 1) tmem_dealloc_pair(tmem_base, GT_TMEM_COLS);
  if (tid == 0 && *abort_flag) atomicCAS(status, 0, misaligned ? TWKV_ERR_DEVICE_CHECK : TWKV_ERR_TIMEOUT);
}

int gate_tc_max_pairs(int sm_count);
size_t gate_tc_stage_bytes(int n_cta, int d) { return (size_t)n_cta * TILE * d * sizeof(unsigned short); }

size_t gate_tc_fix_bytes() { return (size_t)GT_FIX_CAP * 2 * sizeof(int4); }

static cudaError_t launch_gate_fixup(const DevView& v, const GateMaps& maps, const LayerParams& lp, int bf16, unsigned short* levels,
                                     int sm_count, cudaStream_t st) {
  ProfScope ps(TWKV_K_GATE_RANK, st);
  gate_fixup_kernel<<<2 * sm_count, GT_FIX_THREADS, 0, st>>>(maps.raw, bf16, v.d_kv, lp.b_k, lp.b_v, maps.raw.fix_list,
                                                             maps.raw.fix_counters, levels);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_gate_ranks_tc(const DevView& v, const GateMaps& maps, const LayerParams& lp, int n_tok, unsigned short* levels,
                                 int sm_count, bool pairs, cudaStream_t st) {
  if (n_tok <= 0) return cudaSuccess;
  const int d = v.d_kv;
  const int bf16 = v.dtype == TWKV_BF16 ? 1 : 0;
  if (pairs) {
    // maps.wk / maps.wv must have 128-row boxes here (each CTA loads half of a 256-row slab)
    const size_t smem = (size_t)GT2_STAGES * 2 * GT_PANEL_BYTES + TILE * GT_BLK_STRIDE * sizeof(float2) + 8 * (2 * GT2_STAGES + 5) + 16;
    cudaError_t e = cudaFuncSetAttribute(gate_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(GT_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute pair_attr;
    pair_attr.id = cudaLaunchAttributeClusterDimension;
    pair_attr.val.clusterDim.x = 2; pair_attr.val.clusterDim.y = 1; pair_attr.val.clusterDim.z = 1;
    cfg.attrs = &pair_attr;
    cfg.numAttrs = 1;
    const int max_clusters = gate_tc_max_pairs(sm_count);
    if (max_clusters < 1) return cudaErrorInvalidConfiguration;
    const int n_items = 2 * ((n_tok + 2 * TILE - 1) / (2 * TILE));
    cfg.gridDim = dim3(2 * (n_items < max_clusters ? n_items : max_clusters));
    {
      ProfScope ps(TWKV_K_GATE_GEMM, st);
      e = cudaLaunchKernelEx(&cfg, gate_tc2_kernel, maps.xk, maps.xv, maps.wk, maps.wv, lp.b_k, lp.b_v, n_tok, d, bf16, v.tau,
                             v.gate_scratch, levels, v.status, maps.raw);
    }
    count_launch();
    if (e != cudaSuccess) return e;
    return launch_gate_fixup(v, maps, lp, bf16, levels, sm_count, st);
  }
  const int NS = (d % 256 == 0) ? 256 : 128;
  const size_t smem = (size_t)GT_STAGES * (GT_PANEL_BYTES + (size_t)NS * 128) + TILE * GT_BLK_STRIDE * sizeof(float2) + 8 * (2 * GT_STAGES + 5) + 16;
  cudaError_t e = cudaFuncSetAttribute(gate_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int n_items = 2 * ((n_tok + TILE - 1) / TILE);
  const int grid = n_items < sm_count ? n_items : sm_count;
  {
    ProfScope ps(TWKV_K_GATE_GEMM, st);
    gate_tc_kernel<<<grid, GT_THREADS, smem, st>>>(maps.xk, maps.xv, maps.wk, maps.wv, lp.b_k, lp.b_v, n_tok, d, bf16, v.tau,
                                                   v.gate_scratch, levels, v.status, maps.raw);
  }
  count_launch();
  if (cudaError_t e2 = cudaGetLastError(); e2 != cudaSuccess) return e2;
  return launch_gate_fixup(v, maps, lp, bf16, levels, sm_count, st);
}

// CTA pairs of gate_tc2_kernel that can be resident at once on the current device (0: the pair kernel cannot run).
static int gate_tc_query_pairs(int sm_count) {
  const size_t smem = (size_t)GT2_STAGES * 2 * GT_PANEL_BYTES + TILE * GT_BLK_STRIDE * sizeof(float2) + 8 * (2 * GT2_STAGES + 5) + 16;
  if (cudaFuncSetAttribute(gate_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) { cudaGetLastError(); return 0; }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(GT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.gridDim = dim3(sm_count & ~1);
  cudaLaunchAttribute pair_attr;
  pair_attr.id = cudaLaunchAttributeClusterDimension;
  pair_attr.val.clusterDim.x = 2; pair_attr.val.clusterDim.y = 1; pair_attr.val.clusterDim.z = 1;
  cfg.attrs = &pair_attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, gate_tc2_kernel, &cfg) != cudaSuccess || n < 1) { cudaGetLastError(); n = 0; }
  return n;
}
int gate_tc_max_pairs(int sm_count) {
  static const int cached = gate_tc_query_pairs(sm_count);     // queried once per process (thread-safe initialisation)
  return cached;
}

}  // namespace twkv
