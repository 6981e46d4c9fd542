// K-side of decode attention on the 5th-generation tensor cores.
//
// Per K tile (128 tokens of one rank class c, panels [128 x 64] in HBM):
//   Kbar[:, slab g] = X^_K[128 x 64c] . U_K^-1[0:64c, 128g : 128g+128]        (Eq. 3, one KV head at a time)
// is a tcgen05.mma chain (M = 128, N = 128, K = 16 per instruction) whose fp32 accumulator lives in
// TMEM.  Panels of X^_K and of the pre-transposed U_K^-1 arrive by TMA with the 128-byte swizzle,
// which is exactly the K-major operand layout the MMA reads from shared memory.  Two 128-column
// TMEM buffers alternate, so the epilogue of slab g (tcgen05.ld, RoPE by the token's position,
// dot products with the GQA group's queries) overlaps the MMAs of slab g + 1.
//
// Warp roles (320 threads, one CTA per SM, persistent over the class-sorted tile list):
//   warp 0      TMA producer   (X^_K panels into 8 resident slots, U_K^-1 panels into a ring)
//   warp 1      MMA issuer     (one lane issues; owns the TMEM allocation)
//   warps 2-9   epilogue       (thread = one token row x one half of the RoPE frequencies)
// All waits are bounded (tc_util.cuh); a wait that runs out ends the kernel with TWKV_ERR_TIMEOUT.
#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {
using namespace tc;

constexpr int KT_THREADS = 320;
constexpr int KT_EPI = 256;
constexpr int KT_A_SLOTS = 8;
constexpr uint32_t KT_TMEM_COLS = 256;
constexpr uint32_t PANEL_BYTES = 16384;

template <bool BF16> __device__ __forceinline__ float kt_to_f32(unsigned short bits) {
  if constexpr (BF16) return __uint_as_float((unsigned)bits << 16);
  else return __half2float(__ushort_as_half(bits));
}

template <bool BF16, int REP>
__global__ void __launch_bounds__(KT_THREADS, 1)
kscore_tc_kernel(const __grid_constant__ CUtensorMap map_blocks, const __grid_constant__ CUtensorMap map_uinvT,
                 DevView v, int layer, const unsigned short* __restrict__ q, int nb) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ int s_cls_cnt[TWKV_MAX_CLASSES];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hq = v.Hq, Hkv = v.Hkv;
  // carve shared memory; operand tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t raw = smem_addr(smem_raw);
  const uint32_t base_addr = (raw + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base_addr - raw);
  const uint32_t sA = base_addr;
  const uint32_t sB = sA + KT_A_SLOTS * PANEL_BYTES;
  float* sQ = reinterpret_cast<float*>(base_ptr + (KT_A_SLOTS + nb) * PANEL_BYTES);
  float* sS = sQ + Hq * HEAD_DIM;
  const uint32_t bars = smem_addr(sS + TILE * Hq);
  // barrier map (8 bytes each)
  const uint32_t a_full = bars, a_empty = a_full + 8 * KT_A_SLOTS, b_full = a_empty + 8 * KT_A_SLOTS;
  const uint32_t b_empty = b_full + 8 * nb, slab_full = b_empty + 8 * nb, slab_empty = slab_full + 16;
  const uint32_t epi_bar = slab_empty + 16;
  volatile int* abort_flag = &s_abort;

  if (tid == 0) {
    for (int i = 0; i < KT_A_SLOTS; ++i) { mbar_init(a_full + 8 * i, 1); mbar_init(a_empty + 8 * i, 1); }
    for (int i = 0; i < nb; ++i) { mbar_init(b_full + 8 * i, 1); mbar_init(b_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(slab_full + 8 * i, 1); mbar_init(slab_empty + 8 * i, KT_EPI / 32); }
    mbar_init(epi_bar, KT_EPI);
    s_abort = 0;
    mbar_init_fence();
  }
  if (tid < TWKV_MAX_CLASSES) s_cls_cnt[tid] = tid < v.NC ? v.kcc(layer)[tid] : 0;
  if (warp == 1) tmem_alloc(smem_addr(&s_tmem_base), KT_TMEM_COLS);
  for (int i = tid; i < TILE * Hq; i += KT_THREADS) sS[i] = 0.f;
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = s_tmem_base;

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

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) { tma_prefetch_desc(&map_blocks); tma_prefetch_desc(&map_uinvT); }
    uint32_t bk = 0, a_par = 0, a_used = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int cls = dsc.y, blk = dsc.w;
      for (int g = 0; g < Hkv && ok; ++g) {
        for (int j = 0; j < cls && ok; ++j) {
          const int slot = j & (KT_A_SLOTS - 1);
          if (cls > KT_A_SLOTS || g == 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(a_empty + 8 * slot, ((a_par >> slot) & 1u) ^ 1u, abort_flag));
            if (!ok) break;
            if (lane == 0) {
              mbar_expect_tx(a_full + 8 * slot, PANEL_BYTES);
              tma_load_2d(sA + slot * PANEL_BYTES, &map_blocks, a_full + 8 * slot, 0, (blk + j) * TILE);
            }
            a_par ^= 1u << slot;
            a_used |= 1u << slot;
          }
          const uint32_t st = bk % nb, ph = (bk / nb) & 1u;
          ok = __all_sync(0xffffffffu, mbar_wait(b_empty + 8 * st, ph ^ 1u, abort_flag));
          if (!ok) break;
          if (lane == 0) {
            mbar_expect_tx(b_full + 8 * st, PANEL_BYTES);
            tma_load_2d(sB + st * PANEL_BYTES, &map_uinvT, b_full + 8 * st, j * PANEL, g * HEAD_DIM);
          }
          ++bk;
        }
      }
    }
    if (!ok) {
      // give copies already in flight a bounded time to land before the CTA goes away
      for (int i = 0; i < nb; ++i)
        if ((uint32_t)i < bk) mbar_wait_drain(b_full + 8 * i, ((bk - 1 - ((bk - 1 - i) % nb)) / nb) & 1u);
      for (int i = 0; i < KT_A_SLOTS; ++i)
        if ((a_used >> i) & 1u) mbar_wait_drain(a_full + 8 * i, ((a_par >> i) & 1u) ^ 1u);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t idesc = idesc_f16(BF16 ? 1 : 0, 128, 128);
    uint32_t bk = 0, a_par = 0, sc = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int cls = dsc.y;
      for (int g = 0; g < Hkv && ok; ++g) {
        const uint32_t buf = sc & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(slab_empty + 8 * buf, ((sc >> 1) & 1u) ^ 1u, abort_flag));
        if (!ok) break;
        fence_after_sync();
        for (int j = 0; j < cls && ok; ++j) {
          const int slot = j & (KT_A_SLOTS - 1);
          if (cls > KT_A_SLOTS || g == 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(a_full + 8 * slot, (a_par >> slot) & 1u, abort_flag));
            if (!ok) break;
            a_par ^= 1u << slot;
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
              mma_f16_ss(tmem_base + buf * 128, adesc + 2 * ks, bdesc + 2 * ks, idesc, (j > 0 || ks > 0) ? 1u : 0u);
            mma_commit(b_empty + 8 * st);                               // ring stage reusable when these MMAs retire
            if (cls > KT_A_SLOTS || g == Hkv - 1) mma_commit(a_empty + 8 * slot);
            if (j == cls - 1) mma_commit(slab_full + 8 * buf);          // slab accumulator complete
          }
          __syncwarp();
          ++bk;
        }
        ++sc;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int et = tid - 64;
    const int quarter = warp & 3, hf = (warp - 2) >> 2;
    const int row = quarter * 32 + lane;
    uint32_t sc = 0, epar = 0;
    bool ok = true;
    auto epi_sync = [&]() {
      mbar_arrive(epi_bar);
      const bool r = __all_sync(0xffffffffu, mbar_wait(epi_bar, epar, abort_flag));
      epar ^= 1u;
      return r;
    };
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
      int tile, qs; int4 dsc;
      if (!tile_of(w, tile, dsc, qs)) continue;
      const int n_valid = dsc.z;
      for (int i = et; i < Hq * HEAD_DIM; i += KT_EPI)
        sQ[i] = kt_to_f32<BF16>(q[(size_t)qs * Hq * HEAD_DIM + i]) * v.sm_scale;
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
      if (!(ok = epi_sync())) break;
      for (int g = 0; g < Hkv; ++g) {
        const uint32_t buf = sc & 1u;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(slab_full + 8 * buf, (sc >> 1) & 1u, abort_flag)))) break;
        fence_after_sync();
        float lo[32], hi[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * 128 + hf * 32;
        tmem_ld32(taddr, lo);
        tmem_ld32(taddr + 64, hi);
        tmem_ld_wait();
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(slab_empty + 8 * buf);               // TMEM buffer free for slab g + 2
        ++sc;
        float acc[REP];
#pragma unroll
        for (int h = 0; h < REP; ++h) acc[h] = 0.f;
        const float* qg = sQ + (g * REP) * HEAD_DIM + hf * 32;
#pragma unroll
        for (int t = 0; t < 32; ++t) {
          const float y1 = lo[t] * cs[t] - hi[t] * sn[t];
          const float y2 = hi[t] * cs[t] + lo[t] * sn[t];
#pragma unroll
          for (int h = 0; h < REP; ++h) acc[h] += y1 * qg[h * HEAD_DIM + t] + y2 * qg[h * HEAD_DIM + 64 + t];
        }
#pragma unroll
        for (int h = 0; h < REP; ++h) atomicAdd(&sS[row * Hq + g * REP + h], acc[h]);   // two addends per cell: order-independent
      }
      if (!ok) break;
      if (!(ok = epi_sync())) break;
      if (et < Hq) {
        float m = -INFINITY;
        for (int r = 0; r < n_valid; ++r) m = fmaxf(m, sS[r * Hq + et]);
        atomicMax(&v.seqmax[qs * Hq + et], enc_ordered(m));
      }
      if (!(ok = epi_sync())) break;
      float* out = v.scores + (size_t)tile * TILE * Hq;
      for (int i = et; i < TILE * Hq; i += KT_EPI) {
        out[i] = (i / Hq < n_valid) ? sS[i] : -INFINITY;
        sS[i] = 0.f;
      }
    }
  }

  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, KT_TMEM_COLS);
  if (tid == 0 && s_abort) set_status(v, TWKV_ERR_TIMEOUT);
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

size_t kscore_tc_smem_bytes(int Hq, int nb) {
  return 1024 + (size_t)(KT_A_SLOTS + nb) * PANEL_BYTES + (size_t)Hq * HEAD_DIM * 4 + (size_t)TILE * Hq * 4 +
         8 * (2 * KT_A_SLOTS + 2 * nb + 5);
}

template <bool BF16>
static cudaError_t launch_kscore_tc_t(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                                      const void* q, int sm_count, cudaStream_t st) {
  int nb = 4;
  while (nb > 2 && kscore_tc_smem_bytes(v.Hq, nb) > 227 * 1024) --nb;
  const size_t smem = kscore_tc_smem_bytes(v.Hq, nb);
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
