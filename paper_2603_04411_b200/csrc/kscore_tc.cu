// K-side of decode attention on the 5th-generation tensor cores.
//
// Per K tile (128 tokens of one rank class c, panels [128 x 64] in HBM) and per KV head g:
//   Kbar_g = X^_K[128 x 64c] . U_K^-1[0:64c, 128g : 128g+128]                 (Eq. 3)
//   Krot_g = RoPE(Kbar_g, position of each token)                             (keys are rotated after reconstruction)
//   S_g    = Krot_g . Q_g^T,  Q_g = the REP query heads that share KV head g   (the GQA group makes this a dense contraction)
// The first product is a tcgen05.mma chain (M = 128, N = 128, K = 16 per instruction) whose fp32
// accumulator lives in TMEM; X^_K panels and panels of the pre-transposed U_K^-1 arrive by TMA with
// the 128-byte swizzle, which is the K-major operand layout the MMA reads from shared memory.
// Epilogue warps pull the slab out of TMEM, rotate it in fp32, round it to f16 and store it back to
// TMEM, from where it is the A operand of the second product (N = 16, the group's heads padded);
// its accumulator S stays in TMEM until the tile's last slab, so RoPE is the only per-element
// CUDA-core work.  Both sums are linear in X^_K, so a class wider than 8 panels runs as two passes
// over its panels that accumulate into the same S.
//
// Tensor memory (512 columns): slab accumulators 2 x 128 | rotated keys 2 x 64 | S 8 x 16.
// Warp roles (352 threads, one persistent CTA per SM, tiles taken widest class first):
//   warp 0      TMA producer of U_K^-1 panels (ring)
//   warp 1      MMA issuer (one lane issues; owns the TMEM allocation)
//   warps 2-9   epilogue (thread = one token row x one half of the RoPE frequencies)
//   warp 10     TMA producer of X^_K panels (ring of 8 slots, runs ahead into the next tile)
// All waits are bounded (tc_util.cuh); a wait that runs out ends the kernel with TWKV_ERR_TIMEOUT.
//
// Precision: X^_K, U_K^-1 keep the cache dtype with fp32 accumulation; rotated keys and queries enter
// the score product as f16 (keys saturate at +-65504; a bf16 query must be finite in f16).
#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {
using namespace tc;

constexpr int KT_THREADS = 352;
constexpr int KT_EPI = 256;
constexpr int KT_A_SLOTS = 8;
constexpr uint32_t KT_TMEM_COLS = 512;
constexpr uint32_t TM_SLAB = 0, TM_KR = 256, TM_S = 384;      // column offsets inside the allocation
constexpr uint32_t PANEL_BYTES = 16384;
constexpr int KT_Q_ROWS = 72;                                 // 8 rows per KV head + 8 rows of padding
constexpr uint32_t KT_Q_PANEL_BYTES = KT_Q_ROWS * 128;        // one 64-wide K panel of the query operand

template <bool BF16> __device__ __forceinline__ float kt_to_f32(unsigned short bits) {
  if constexpr (BF16) return __uint_as_float((unsigned)bits << 16);
  else return __half2float(__ushort_as_half(bits));
}

template <int N> __device__ __forceinline__ void tmem_ldN(uint32_t taddr, uint32_t* r) {
  if constexpr (N == 1) tmem_ld1(taddr, r);
  else if constexpr (N == 2) tmem_ld2(taddr, r);
  else if constexpr (N == 4) tmem_ld4(taddr, r);
  else tmem_ld8(taddr, r);
}

template <bool BF16, int REP>
__global__ void __launch_bounds__(KT_THREADS, 1)
kscore_tc_kernel(const __grid_constant__ CUtensorMap map_blocks, const __grid_constant__ CUtensorMap map_uinvT,
                 DevView v, int layer, const unsigned short* __restrict__ q, int nb) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hq = v.Hq, Hkv = v.Hkv;
  // operand tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t sA = smem_addr(smem_raw);
  if (sA & 1023u) {
    if (tid == 0) set_status(v, TWKV_ERR_DEVICE_CHECK);
    return;
  }
  const uint32_t sB = sA + KT_A_SLOTS * PANEL_BYTES;
  const uint32_t sQ = sB + nb * PANEL_BYTES;
  unsigned char* sQ_ptr = smem_raw + (KT_A_SLOTS + nb) * PANEL_BYTES;
  unsigned char* tail = sQ_ptr + 2 * KT_Q_PANEL_BYTES;
  const uint32_t bars = smem_addr(tail);
  // barrier map (8 bytes each)
  const uint32_t a_full = bars, a_empty = a_full + 8 * KT_A_SLOTS, b_full = a_empty + 8 * KT_A_SLOTS;
  const uint32_t b_empty = b_full + 8 * nb, slab_full = b_empty + 8 * nb, slab_empty = slab_full + 16;
  const uint32_t kr_full = slab_empty + 16, kr_empty = kr_full + 16, s_full = kr_empty + 16;
  int* s_cls_cnt = reinterpret_cast<int*>(tail + 8 * (2 * KT_A_SLOTS + 2 * nb + 9));
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(s_cls_cnt + TWKV_MAX_CLASSES);
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  if (tid == 0) {
    for (int i = 0; i < KT_A_SLOTS; ++i) { mbar_init(a_full + 8 * i, 1); mbar_init(a_empty + 8 * i, 1); }
    for (int i = 0; i < nb; ++i) { mbar_init(b_full + 8 * i, 1); mbar_init(b_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(slab_full + 8 * i, 1); mbar_init(slab_empty + 8 * i, KT_EPI / 32);
      mbar_init(kr_full + 8 * i, KT_EPI / 32); mbar_init(kr_empty + 8 * i, 1);
    }
    mbar_init(s_full, 1);
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (tid < TWKV_MAX_CLASSES) s_cls_cnt[tid] = tid < v.NC ? v.kcc(layer)[tid] : 0;
  if (warp == 1) tmem_alloc(smem_addr(s_tmem_base), KT_TMEM_COLS);
  for (int i = tid; i < 2 * (int)KT_Q_PANEL_BYTES / 16; i += KT_THREADS)        // padding rows of the query operand stay zero
    reinterpret_cast<uint4*>(sQ_ptr)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  int total = 0;
  for (int c = 0; c < v.NC; ++c) total += s_cls_cnt[c];
  const int4* desc = v.desc(layer, 0);
  const int* kct = v.kct(layer);

  // tile w of the class-sorted list (widest class first) -> (tile id, descriptor); false if not decoded now
  auto tile_of = [&](int w, int& tile, int4& dsc, int& qs) {
    int cls = v.NC, idx = w;
    while (idx >= s_cls_cnt[cls - 1]) { idx -= s_cls_cnt[cls - 1]; --cls; }
    tile = kct[(size_t)(cls - 1) * v.NT + idx];
    dsc = desc[tile];
    qs = v.qslot[dsc.x];
    return qs >= 0;
  };

  if (warp == 10) {
    // ------------------------------------------------------------- TMA producer: X^_K panels
    if (lane == 0) tma_prefetch_desc(&map_blocks);
    uint32_t ak = 0;                                            // panels loaded so far; slot = ak % 8
    bool ok = true;
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int cls = dsc.y, blk = dsc.w;
      for (int j = 0; j < cls && ok; ++j, ++ak) {
        const uint32_t slot = ak % KT_A_SLOTS, ph = (ak / KT_A_SLOTS) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(a_empty + 8 * slot, ph ^ 1u, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(a_full + 8 * slot, PANEL_BYTES);
          tma_load_2d(sA + slot * PANEL_BYTES, &map_blocks, a_full + 8 * slot, 0, (blk + j) * TILE);
        }
      }
    }
    if (!ok)                                                    // let copies in flight land before the CTA goes away
      for (uint32_t i = 0; i < (uint32_t)KT_A_SLOTS && i < ak; ++i) {
        const uint32_t n = ak - 1 - i;
        mbar_wait_drain(a_full + 8 * (n % KT_A_SLOTS), (n / KT_A_SLOTS) & 1u);
      }
  } else if (warp == 0) {
    // ------------------------------------------------------------- TMA producer: U_K^-1 panels
    if (lane == 0) tma_prefetch_desc(&map_uinvT);
    uint32_t bk = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int cls = dsc.y;
      for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
        const int np = min(KT_A_SLOTS, cls - p0);
        for (int g = 0; g < Hkv && ok; ++g) {
          for (int j = 0; j < np && ok; ++j, ++bk) {
            const uint32_t st = bk % nb, ph = (bk / nb) & 1u;
            ok = __all_sync(0xffffffffu, mbar_wait(b_empty + 8 * st, ph ^ 1u, abort_flag));
            if (!ok) break;
            if (lane == 0) {
              mbar_expect_tx(b_full + 8 * st, PANEL_BYTES);
              tma_load_2d(sB + st * PANEL_BYTES, &map_uinvT, b_full + 8 * st, (p0 + j) * PANEL, g * HEAD_DIM);
            }
          }
        }
      }
    }
    if (!ok)
      for (uint32_t i = 0; i < (uint32_t)nb && i < bk; ++i) {
        const uint32_t n = bk - 1 - i;
        mbar_wait_drain(b_full + 8 * (n % nb), (n / nb) & 1u);
      }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    const uint32_t idesc_main = idesc_f16(BF16 ? 1 : 0, 128, 128);
    const uint32_t idesc_s = idesc_f16(0, 128, 16);
    uint32_t bk = 0, ak = 0, sc = 0;
    bool ok = true;
    // the score product of slab n is issued after the main product of slab n + 1, so the tensor
    // pipe has work while the epilogue warps rotate slab n
    bool pend = false, pend_acc = false, pend_last = false;
    uint32_t pend_sc = 0; int pend_g = 0;
    auto issue_scores = [&]() {
      const uint32_t kb = pend_sc & 1u;
      if (!__all_sync(0xffffffffu, mbar_wait(kr_full + 8 * kb, (pend_sc >> 1) & 1u, abort_flag))) return false;
      fence_after_sync();
      if (lane == 0) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t qdesc = kmajor_sw128_desc(sQ + (ks >> 2) * KT_Q_PANEL_BYTES + pend_g * 1024) + 2 * (ks & 3);
          mma_f16_ts(tmem_base + TM_S + 16 * pend_g, tmem_base + TM_KR + 64 * kb + 8 * ks, qdesc, idesc_s,
                     (pend_acc || ks > 0) ? 1u : 0u);
        }
        mma_commit(kr_empty + 8 * kb);
        if (pend_last) mma_commit(s_full);
      }
      __syncwarp();
      pend = false;
      return true;
    };
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int cls = dsc.y;
      for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
        const int np = min(KT_A_SLOTS, cls - p0);
        for (int g = 0; g < Hkv && ok; ++g) {
          const uint32_t buf = sc & 1u;
          ok = __all_sync(0xffffffffu, mbar_wait(slab_empty + 8 * buf, ((sc >> 1) & 1u) ^ 1u, abort_flag));
          if (!ok) break;
          fence_after_sync();
          for (int j = 0; j < np && ok; ++j, ++bk) {
            const uint32_t an = ak + j, slot = an % KT_A_SLOTS;
            if (g == 0) {
              ok = __all_sync(0xffffffffu, mbar_wait(a_full + 8 * slot, (an / KT_A_SLOTS) & 1u, abort_flag));
              if (!ok) break;
            }
            const uint32_t st = bk % nb, ph = (bk / nb) & 1u;
            ok = __all_sync(0xffffffffu, mbar_wait(b_full + 8 * st, ph, abort_flag));
            if (!ok) break;
            fence_after_sync();
            if (lane == 0) {
              const uint64_t adesc = kmajor_sw128_desc(sA + slot * PANEL_BYTES);
              const uint64_t bdesc = kmajor_sw128_desc(sB + st * PANEL_BYTES);
#pragma unroll
              for (int ks = 0; ks < 4; ++ks)
                mma_f16_ss(tmem_base + TM_SLAB + buf * 128, adesc + 2 * ks, bdesc + 2 * ks, idesc_main, (j > 0 || ks > 0) ? 1u : 0u);
              mma_commit(b_empty + 8 * st);                             // ring stage reusable when these MMAs retire
              if (g == Hkv - 1) mma_commit(a_empty + 8 * slot);         // last slab of the pass: the X^_K panel is done
              if (j == np - 1) mma_commit(slab_full + 8 * buf);         // slab accumulator complete
            }
            __syncwarp();
          }
          if (!ok) break;
          if (pend && !(ok = issue_scores())) break;
          pend = true; pend_sc = sc; pend_g = g; pend_acc = p0 > 0; pend_last = (p0 + np >= cls) && (g == Hkv - 1);
          ++sc;
        }
        ak += np;
      }
    }
    if (ok && pend) issue_scores();
  } else {
    // ------------------------------------------------------------- epilogue
    const int et = tid - 64;
    const int quarter = warp & 3, hf = (warp - 2) >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int g_lo = hf ? (Hkv + 1) / 2 : 0, g_hi = hf ? Hkv : (Hkv + 1) / 2;
    uint32_t sc = 0, tcount = 0;
    int prev_qs = -1;
    bool ok = true;
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int cls = dsc.y, n_valid = dsc.z;
      if (qs != prev_qs) {
        // the group's queries as the K-major, 128-byte-swizzled B operand: row 8 g + h, two 64-wide panels.
        // The previous tile's score products have retired (s_full was waited for), so the rows are free.
        for (int i = et; i < Hq * 16; i += KT_EPI) {
          const int head = i >> 4, ch = i & 15;                               // 8 dims per chunk
          const uint4 raw = *reinterpret_cast<const uint4*>(q + ((size_t)qs * Hq + head) * HEAD_DIM + ch * 8);
          uint4 val = raw;
          if constexpr (BF16) {
            const unsigned short* e = reinterpret_cast<const unsigned short*>(&raw);
            val.x = pack_f16x2_sat(kt_to_f32<true>(e[0]), kt_to_f32<true>(e[1]));
            val.y = pack_f16x2_sat(kt_to_f32<true>(e[2]), kt_to_f32<true>(e[3]));
            val.z = pack_f16x2_sat(kt_to_f32<true>(e[4]), kt_to_f32<true>(e[5]));
            val.w = pack_f16x2_sat(kt_to_f32<true>(e[6]), kt_to_f32<true>(e[7]));
          }
          const int qrow = (head / REP) * 8 + head % REP, c8 = ch & 7;
          *reinterpret_cast<uint4*>(sQ_ptr + (ch >> 3) * KT_Q_PANEL_BYTES + qrow * 128 + ((c8 ^ (qrow & 7)) << 4)) = val;
        }
        fence_proxy_async_smem();
        prev_qs = qs;
      }
      float cs[32], sn[32];
      {
        const int pos = v.aux(layer, 0)[(size_t)tile * TILE + row];
        const float2* th = v.rope_hi + (size_t)((pos >> 9) & (ROPE_HI - 1)) * 64 + hf * 32;
        const float2* tl = v.rope_lo + (size_t)(pos & (ROPE_LO - 1)) * 64 + hf * 32;
#pragma unroll
        for (int t = 0; t < 32; ++t) {
          const float2 a = th[t], b = tl[t];
          cs[t] = a.x * b.x - a.y * b.y;
          sn[t] = a.y * b.x + a.x * b.y;
        }
      }
      const int n_slabs = ((cls + KT_A_SLOTS - 1) / KT_A_SLOTS) * Hkv;
      for (int sl = 0; sl < n_slabs; ++sl, ++sc) {
        const uint32_t buf = sc & 1u, par = (sc >> 1) & 1u;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(slab_full + 8 * buf, par, abort_flag)))) break;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(kr_empty + 8 * buf, par ^ 1u, abort_flag)))) break;
        fence_after_sync();
        const uint32_t slab = lane_addr + TM_SLAB + buf * 128 + hf * 32;
        const uint32_t kr = lane_addr + TM_KR + buf * 64 + hf * 16;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          float lo[16], hi[16];
          tmem_ld16(slab + half * 16, reinterpret_cast<uint32_t*>(lo));
          tmem_ld16(slab + 64 + half * 16, reinterpret_cast<uint32_t*>(hi));
          tmem_ld_wait();
          if (half == 1) {                                                  // the slab accumulator is free for slab n + 2
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(slab_empty + 8 * buf);
          }
          uint32_t p1[8], p2[8];
#pragma unroll
          for (int t = 0; t < 16; t += 2) {
            const float c0 = cs[half * 16 + t], s0 = sn[half * 16 + t], c1 = cs[half * 16 + t + 1], s1 = sn[half * 16 + t + 1];
            p1[t >> 1] = pack_f16x2_sat(lo[t] * c0 - hi[t] * s0, lo[t + 1] * c1 - hi[t + 1] * s1);
            p2[t >> 1] = pack_f16x2_sat(hi[t] * c0 + lo[t] * s0, hi[t + 1] * c1 + lo[t + 1] * s1);
          }
          tmem_st8(kr + half * 8, p1);                                      // dims d -> column d / 2
          tmem_st8(kr + 32 + half * 8, p2);                                 // dims 64 + d
        }
        tmem_st_wait();
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(kr_full + 8 * buf);
      }
      if (!ok) break;
      // all score products of the tile have retired: scale, mask the rows past the last token, store
      if (!(ok = __all_sync(0xffffffffu, mbar_wait(s_full, tcount & 1u, abort_flag)))) break;
      ++tcount;
      fence_after_sync();
      float* out = v.scores + ((size_t)tile * TILE + row) * Hq;
      for (int g = g_lo; g < g_hi; ++g) {
        float s[REP];
        tmem_ldN<REP>(lane_addr + TM_S + 16 * g, reinterpret_cast<uint32_t*>(s));
        tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < REP; ++h) s[h] = row < n_valid ? s[h] * v.sm_scale : -INFINITY;
        if constexpr (REP == 1) out[g] = s[0];
        else if constexpr (REP == 2) *reinterpret_cast<float2*>(out + g * 2) = make_float2(s[0], s[1]);
        else {
#pragma unroll
          for (int h = 0; h < REP; h += 4) *reinterpret_cast<float4*>(out + g * REP + h) = make_float4(s[h], s[h + 1], s[h + 2], s[h + 3]);
        }
#pragma unroll
        for (int h = 0; h < REP; ++h) {
          float m = s[h];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          if (lane == 0) atomicMax(&v.seqmax[qs * Hq + g * REP + h], enc_ordered(m));
        }
      }
    }
  }

  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, KT_TMEM_COLS);
  if (tid == 0 && *abort_flag) set_status(v, TWKV_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// [rows][cols] 16-bit row-major -> transposed copy; used once per layer to make U_K^-1 (and the
// gate weights) K-major for the tensor cores.
__global__ void transpose16_kernel(const unsigned short* __restrict__ in, unsigned short* __restrict__ out, int n) {
  __shared__ unsigned short t[32][33];
  const int bx = blockIdx.x * 32, by = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) t[r][threadIdx.x] = in[(size_t)(by + r) * n + bx + threadIdx.x];
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) out[(size_t)(bx + r) * n + by + threadIdx.x] = t[threadIdx.x][r];
}

cudaError_t launch_transpose16(const void* in, void* out, int n, cudaStream_t st) {
  ProfScope ps(TWKV_K_OTHER, st);
  transpose16_kernel<<<dim3(n / 32, n / 32), dim3(32, 8), 0, st>>>(reinterpret_cast<const unsigned short*>(in),
                                                                    reinterpret_cast<unsigned short*>(out), n);
  count_launch();
  return cudaGetLastError();
}

size_t kscore_tc_smem_bytes(int nb) {
  return (size_t)(KT_A_SLOTS + nb) * PANEL_BYTES + 2 * KT_Q_PANEL_BYTES + 8 * (2 * KT_A_SLOTS + 2 * nb + 9) +
         (TWKV_MAX_CLASSES + 2) * sizeof(int);
}

template <bool BF16>
static cudaError_t launch_kscore_tc_t(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                                      const void* q, int sm_count, cudaStream_t st) {
  int nb = 5;
  while (nb > 2 && kscore_tc_smem_bytes(nb) > 227 * 1024) --nb;
  const size_t smem = kscore_tc_smem_bytes(nb);
  const unsigned short* qq = reinterpret_cast<const unsigned short*>(q);
  ProfScope ps(TWKV_K_KSCORE, st);
#define TWKV_KT(REP)                                                                                                  \
  {                                                                                                                   \
    cudaError_t e = cudaFuncSetAttribute(kscore_tc_kernel<BF16, REP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                                   \
    kscore_tc_kernel<BF16, REP><<<sm_count, KT_THREADS, smem, st>>>(map_blocks, map_uinvT, v, layer, qq, nb);         \
  }
  switch (v.rep) {
    case 1: TWKV_KT(1) break;
    case 2: TWKV_KT(2) break;
    case 4: TWKV_KT(4) break;
    default: TWKV_KT(8) break;
  }
#undef TWKV_KT
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_kscore_tc(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                             const void* q, int sm_count, cudaStream_t st) {
  return v.dtype == TWKV_BF16 ? launch_kscore_tc_t<true>(v, layer, map_blocks, map_uinvT, q, sm_count, st)
                              : launch_kscore_tc_t<false>(v, layer, map_blocks, map_uinvT, q, sm_count, st);
}

}  // namespace twkv
