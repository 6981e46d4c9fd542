// K-side of decode attention on the 5th-generation tensor cores.
//
// Per K tile (128 tokens of one rank class c, panels [128 x 64] in HBM) and per KV head g:
//   Kbar_g = X^_K[128 x 64c] . U_K^-1[0:64c, 128g : 128g+128]                 (Eq. 3)
//   Krot_g = RoPE(Kbar_g, position of each token)                             (keys are rotated after reconstruction)
//   S_g    = Krot_g . Q_g^T,  Q_g = the REP query heads that share KV head g   (the GQA group makes this a dense contraction)
// The first product is a tcgen05.mma chain (M = 128, N = 128, K = 16 per instruction) whose fp32
// accumulator (a "slab") lives in TMEM; X^_K panels and panels of U_K^-1 (re-tiled once per layer into contiguous
// [128 x 64] transposed panels) arrive by TMA with the 128-byte swizzle, which is the K-major operand layout the MMA
// reads from shared memory.
// Epilogue warps pull the slab out of TMEM sixteen columns at a time, rotate it in fp32, split every value into a
// high and a low f16 part and store both back IN PLACE (a thread overwrites only columns it has already read: 64
// fp32 columns become 32 columns of high parts and 32 of low parts), from where they are the A operands of the second
// product (N = 16, the group's heads padded; one product per part).  The order of the 128 dimensions along the
// contraction is whatever that in-place layout gives; the query operand is written in the same order.
// Each slab's scores land in one of four 16-column accumulators and are read out by the epilogue warps two slabs
// later (scaled, masked, stored, folded into the per-(sequence, head) maximum), so that a tile has no tail:
// RoPE is the only per-element CUDA-core work.  Both products are linear in X^_K, so a class wider than 8 panels runs
// as two passes over its panels; the second pass adds to the scores the first one stored.
//
// Tensor memory (512 columns): slabs 3 x 128 | score accumulators 4 x 16.
// Warp roles (384 threads, one persistent CTA per SM working through a contiguous, cost-balanced piece of the tile list):
//   warp 0      TMA producer of U_K^-1 panels (ring, one lane per stage)
//   warp 1      issuer of the main products (one elected lane; owns the TMEM allocation)
//   warps 2-9   epilogue (thread = one token row x one half of the RoPE frequencies)
//   warp 10     TMA producer of X^_K panels (ring of 8 slots served by four lanes, runs ahead into the next tiles)
//   warp 11     issuer of the score products (one elected lane)
// A slab buffer goes round: main products (slab_full) -> epilogue (kr_full) -> score products (slab_empty).
// All waits are bounded (tc_util.cuh); a wait that runs out ends the kernel with TWKV_ERR_TIMEOUT.
//
// Precision: X^_K, U_K^-1 keep the cache dtype with fp32 accumulation; queries enter the score product as
// f16 (a bf16 query must be finite in f16), rotated keys as the sum of two f16 (21 significant bits; they
// saturate at +-65504).
#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {
using namespace tc;

constexpr int KT_THREADS = 384;
constexpr int KT_EPI = 256;
constexpr int KT_A_SLOTS = 8;                                  // power of two (slot = panel count & 7, phase = bit 3)
constexpr int KT_SLABS = 3;                                    // slab buffers
constexpr int KT_S_SLOTS = 4;                                  // score accumulators
constexpr uint32_t KT_TMEM_COLS = 512;
constexpr uint32_t TM_SLAB = 0, TM_S = 128 * KT_SLABS;        // column offsets inside the allocation
constexpr uint32_t PANEL_BYTES = 16384;
constexpr int KT_Q_ROWS = 72;                                 // 8 rows per KV head + 8 rows of padding
constexpr uint32_t KT_Q_PANEL_BYTES = KT_Q_ROWS * 128;        // one 64-wide K panel of the query operand
constexpr int KT_ROPE_STRIDE = 33;                            // float4 per row of the small RoPE table in shared memory (32 + 1 against bank conflicts)
constexpr uint32_t KT_ROPE_STAGE_BYTES = ROPE_LO * KT_ROPE_STRIDE * 16;
constexpr int KT_HOT_PANELS = 4;                              // panel rows of U_K^-1 (64 spectral components each) kept in several copies
constexpr int KT_UINV_COPIES = 8;
constexpr int KT_N_BARS = 2 * KT_A_SLOTS + 3 * KT_SLABS + 2 * KT_S_SLOTS;     // + 2 nb for the U_K^-1 ring

// Packed fp32 pairs (two lanes per 64-bit register, one instruction for both): the rotation is issue-bound.
__device__ __forceinline__ uint64_t f2_pack(float a, float b) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ uint64_t f2_pack_bits(uint32_t a, uint32_t b) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b)); return r; }
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) { uint64_t r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) { uint64_t r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) { uint64_t r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
__device__ __forceinline__ uint32_t f2_to_f16x2_sat(uint64_t v) {       // (lo lane -> bits 0..15), saturating
  uint32_t d;
  asm("{\n\t.reg .f32 a, b;\n\tmov.b64 {a, b}, %1;\n\tcvt.rn.satfinite.f16x2.f32 %0, b, a;\n\t}" : "=r"(d) : "l"(v));
  return d;
}
__device__ __forceinline__ unsigned warp_max_u32(unsigned x) {
  unsigned r;
  asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(x));
  return r;
}

template <bool BF16> __device__ __forceinline__ float kt_to_f32(unsigned short bits) {
  if constexpr (BF16) return __uint_as_float((unsigned)bits << 16);
  else return __half2float(__ushort_as_half(bits));
}

// A score read-out that is still owed: which accumulator, where the scores go, how they combine.
struct KtPending {
  float* out;            // this thread's row of the score scratch, at the group's first head
  int mxi;               // which of the reading thread's running maxima the scores fold into (slab index / 2)
  uint32_t meta;         // bit 0 valid | bit 1 reader half | bits 2-3 mode | bits 4-5 accumulator | bit 6 its parity | bit 7 row is a token
};
constexpr uint32_t KP_VALID = 1u, KP_LIVE = 128u;
constexpr uint32_t KP_STORE_PART = 0u, KP_STORE_FINAL = 1u, KP_ADD_FINAL = 2u;      // modes

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
  float4* sRope = reinterpret_cast<float4*>(sQ_ptr + 2 * KT_Q_PANEL_BYTES);   // [16 rows][33]: the small RoPE table
  unsigned char* tail = sQ_ptr + 2 * KT_Q_PANEL_BYTES + KT_ROPE_STAGE_BYTES;
  const uint32_t bars = smem_addr(tail);
  // barrier map (8 bytes each)
  const uint32_t a_full = bars, a_empty = a_full + 8 * KT_A_SLOTS, b_full = a_empty + 8 * KT_A_SLOTS;
  const uint32_t b_empty = b_full + 8 * nb, slab_full = b_empty + 8 * nb, kr_full = slab_full + 8 * KT_SLABS;
  const uint32_t slab_empty = kr_full + 8 * KT_SLABS, s_full = slab_empty + 8 * KT_SLABS, s_empty = s_full + 8 * KT_S_SLOTS;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (KT_N_BARS + 2 * nb));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  if (tid == 0) {
    for (int i = 0; i < KT_A_SLOTS; ++i) { mbar_init(a_full + 8 * i, 1); mbar_init(a_empty + 8 * i, 1); }
    for (int i = 0; i < nb; ++i) { mbar_init(b_full + 8 * i, 1); mbar_init(b_empty + 8 * i, 1); }
    for (int i = 0; i < KT_SLABS; ++i) {
      mbar_init(slab_full + 8 * i, 1); mbar_init(kr_full + 8 * i, KT_EPI / 32); mbar_init(slab_empty + 8 * i, 1);
    }
    for (int i = 0; i < KT_S_SLOTS; ++i) { mbar_init(s_full + 8 * i, 1); mbar_init(s_empty + 8 * i, KT_EPI / 64); }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(smem_addr(s_tmem_base), KT_TMEM_COLS);
  for (int i = tid; i < 2 * (int)KT_Q_PANEL_BYTES / 16; i += KT_THREADS)        // padding rows of the query operand stay zero
    reinterpret_cast<uint4*>(sQ_ptr)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = tid; i < ROPE_LO * 32; i += KT_THREADS) sRope[(i >> 5) * KT_ROPE_STRIDE + (i & 31)] = v.rope_lo[i];
  fence_proxy_async_smem();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // work list written by plan_kernel: the K tiles of the sequences being decoded, widest class first
  // this CTA's contiguous piece [w0, total) of the list (cut by estimated cost)
  const int w0 = v.cta_start[blockIdx.x], total = v.cta_start[blockIdx.x + 1];
  const int4* klist = v.klist;
  const int4 kt_none = make_int4(0, 0, 0, -1);
  // CTAs walk the KV heads in rotated order, so that at any moment they read different panels of U_K^-1 from L2
  const int g_rot = blockIdx.x % Hkv;

  if (warp == 10) {
    // ------------------------------------------------------------- TMA producer: X^_K panels
    // A thread's TMA copies complete one after the other, so the ring is served by four lanes (lane L issues the
    // copies of slots L and L + 4) that each keep their own copy in flight.  The four lanes walk the panel sequence
    // together and wait on the same barrier (slots free up in order): lanes of one warp blocked on different barriers
    // would run one after the other, each one's wait holding up the others' copies.
    if (lane < 4) {
      if (lane == 0) tma_prefetch_desc(&map_blocks);
      uint32_t ak = 0;                                          // panels so far; slot = ak % 8
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[w + 1] : kt_none;
        const int cls = e.y & 0xff, blk = e.z;
        for (int j = 0; j < cls; ++j, ++ak) {
          const uint32_t slot = ak % KT_A_SLOTS, ph = (ak / KT_A_SLOTS) & 1u;
          if (!(ok = __all_sync(0xfu, mbar_wait(a_empty + 8 * slot, ph ^ 1u, abort_flag)))) break;
          if ((slot & 3u) == (uint32_t)lane) {
            mbar_expect_tx(a_full + 8 * slot, PANEL_BYTES);
            tma_load_2d(sA + slot * PANEL_BYTES, &map_blocks, a_full + 8 * slot, 0, (blk + j) * TILE);
          }
          __syncwarp(0xfu);
        }
        e = nxt;
      }
      if (!ok)                                                  // let copies in flight land before the CTA goes away
        for (uint32_t i = 0; i < (uint32_t)KT_A_SLOTS && i < ak; ++i) {
          const uint32_t n = ak - 1 - i;
          if (((n % KT_A_SLOTS) & 3u) == (uint32_t)lane) mbar_wait_drain(a_full + 8 * (n % KT_A_SLOTS), (n / KT_A_SLOTS) & 1u);
        }
    }
    __syncwarp();
  } else if (warp == 0) {
    // ------------------------------------------------------------- TMA producer: U_K^-1 panels
    // one lane per ring stage, walking the panel sequence together, for the same reasons
    if (lane < nb) {
      const unsigned lanes = (1u << nb) - 1u;
      if (lane == 0) tma_prefetch_desc(&map_uinvT);
      uint32_t bk = 0, bst = 0, bph = 0;                        // panels so far; ring stage and its phase
      bool ok = true;
      // this CTA's copy of the hot panel rows (copy 0 is the full matrix itself)
      const int hot_copy = (blockIdx.x / Hkv) % KT_UINV_COPIES;
      const int hot_base = v.NC * Hkv + (hot_copy - 1) * KT_HOT_PANELS * Hkv;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[w + 1] : kt_none;
        const int cls = e.y & 0xff;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const int np = min(KT_A_SLOTS, cls - p0);
          for (int sl = 0; sl < Hkv && ok; ++sl) {
            const int g = sl + g_rot < Hkv ? sl + g_rot : sl + g_rot - Hkv;
            for (int j = 0; j < np; ++j, ++bk) {
              const uint32_t st = bst, ph = bph;
              if (++bst == (uint32_t)nb) { bst = 0; bph ^= 1u; }
              if (!(ok = __all_sync(lanes, mbar_wait(b_empty + 8 * st, ph ^ 1u, abort_flag)))) break;
              if (st == (uint32_t)lane) {
                const int pj = p0 + j;
                const int prow = pj < KT_HOT_PANELS && hot_copy ? hot_base + pj * Hkv + g : pj * Hkv + g;     // panel index in the re-tiled copy
                mbar_expect_tx(b_full + 8 * st, PANEL_BYTES);
                tma_load_2d(sB + st * PANEL_BYTES, &map_uinvT, b_full + 8 * st, 0, prow * HEAD_DIM);
              }
              __syncwarp(lanes);
            }
          }
        }
        e = nxt;
      }
      if (!ok)
        for (uint32_t i = 0; i < (uint32_t)nb && i < bk; ++i) {
          const uint32_t n = bk - 1 - i;
          if (n % nb == (uint32_t)lane) mbar_wait_drain(b_full + 8 * (n % nb), (n / nb) & 1u);
        }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (one elected lane runs the whole role)
    if (elect_one()) {
      // This role is one thread issuing asynchronous work; what it costs is its own instruction stream (a 64-cycle MMA
      // per few instructions), so descriptors are stepped with 32-bit adds, a panel's four MMAs are one asm block, and
      // every wait tries once inline before it falls into the bounded loop.
      const uint32_t idesc_main = idesc_f16(BF16 ? 1 : 0, 128, 128);
      const uint32_t a_lo0 = kmajor_sw128_desc_lo(sA), b_lo0 = kmajor_sw128_desc_lo(sB);
      uint32_t bst = 0, bph = 0, ak = 0, sbuf = 0, sph = 0;
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[w + 1] : kt_none;
        const int cls = e.y & 0xff;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const int np = min(KT_A_SLOTS, cls - p0);
          for (int sl = 0; sl < Hkv && ok; ++sl) {
            // the buffer is free once the score products over its previous contents have retired
            if (!(ok = mbar_wait_thin(slab_empty + 8 * sbuf, sph ^ 1u, abort_flag))) break;
            fence_after_sync();
            const uint32_t d = tmem_base + TM_SLAB + sbuf * 128;
            const bool first = sl == 0, last = sl == Hkv - 1;
            uint32_t an = ak;
            for (int j = 0; j < np; ++j, ++an) {
              const uint32_t slot = an & (KT_A_SLOTS - 1);
              if (first && !(ok = mbar_wait_thin(a_full + 8 * slot, (an >> 3) & 1u, abort_flag))) break;
              const uint32_t st = bst;
              if (!(ok = mbar_wait_thin(b_full + 8 * st, bph, abort_flag))) break;
              if (++bst == (uint32_t)nb) { bst = 0; bph ^= 1u; }
              fence_after_sync();
              mma_f16_ss_panel(d, a_lo0 + slot * (PANEL_BYTES >> 4), b_lo0 + st * (PANEL_BYTES >> 4), idesc_main, j > 0 ? 1u : 0u);
              mma_commit(b_empty + 8 * st);                             // ring stage reusable when these MMAs retire
              if (last) mma_commit(a_empty + 8 * slot);                 // last slab of the pass: the X^_K panel is done
            }
            if (!ok) break;
            mma_commit(slab_full + 8 * sbuf);                           // slab accumulator complete
            if (++sbuf == (uint32_t)KT_SLABS) { sbuf = 0; sph ^= 1u; }
          }
          ak += np;
        }
        e = nxt;
      }
    }
    __syncwarp();
  } else if (warp == 11) {
    // ------------------------------------------------------------- score-product issuer (one elected lane)
    // S (+)= Krot_g . Q_g^T as soon as the epilogue warps have stored a rotated slab; a thread of its own, so that
    // neither issue stream waits for the other's barriers
    if (elect_one()) {
      const uint32_t idesc_s = idesc_f16(0, 128, 16);
      const uint32_t q_lo0 = kmajor_sw128_desc_lo(sQ);
      uint32_t sbuf = 0, sph = 0, slot = 0, slph = 0;
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[w + 1] : kt_none;
        const int cls = e.y & 0xff;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          for (int sl = 0; sl < Hkv; ++sl) {
            const int g = sl + g_rot < Hkv ? sl + g_rot : sl + g_rot - Hkv;
            if (!(ok = mbar_wait_thin(kr_full + 8 * sbuf, sph, abort_flag))) break;
            if (!(ok = mbar_wait_thin(s_empty + 8 * slot, slph ^ 1u, abort_flag))) break;
            fence_after_sync();
            // the rotated keys come as a high and a low f16 part (their sum carries 21 bits): two products into the same S
            const uint32_t kr = tmem_base + TM_SLAB + sbuf * 128, sd = tmem_base + TM_S + 16 * slot;
            mma_f16_ts_k128(sd, kr, q_lo0 + g * (1024 >> 4), KT_Q_PANEL_BYTES >> 4, idesc_s, 0u);
            mma_f16_ts_k128(sd, kr + 64, q_lo0 + g * (1024 >> 4), KT_Q_PANEL_BYTES >> 4, idesc_s, 1u);
            mma_commit(slab_empty + 8 * sbuf);                          // the slab buffer may be overwritten
            mma_commit(s_full + 8 * slot);                              // this slab's scores are complete
            if (++sbuf == (uint32_t)KT_SLABS) { sbuf = 0; sph ^= 1u; }
            if (++slot == (uint32_t)KT_S_SLOTS) { slot = 0; slph ^= 1u; }
          }
        }
        e = nxt;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------- epilogue
    const int et = tid - 64;
    const int quarter = warp & 3, hf = (warp - 2) >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float sm_scale = v.sm_scale;
    const int* kpos = v.aux(layer, 0);
    const float4* __restrict__ rope_hi = v.rope_hi;
    uint32_t sbuf = 0, sph = 0, slot = 0, slph = 0;
    bool ok = true;
    uint64_t cs2[16], sn2[16];                                    // the tile's rotation factors, frequencies (2 t, 2 t + 1) packed
    float tmax[4][REP];                                           // running maxima of the heads this thread reads out (slab index / 2)
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int i = 0; i < REP; ++i) tmax[a][i] = -INFINITY;

    // cos / sin of (row, frequency): pos = hi * 16 + lo, the two table rows combine by the angle-addition formulas.
    // The lo row comes from shared memory (padded rows: lanes with different rows hit different banks), the hi row
    // from global memory (L2; neighbouring positions share it).
    auto rope_setup = [&](int pos) {
      const float4* __restrict__ th = rope_hi + (size_t)((pos >> 4) & (ROPE_HI - 1)) * 32 + hf * 16;
      const float4* tl = sRope + (pos & 15) * KT_ROPE_STRIDE + hf * 16;
      float4 h[16];
#pragma unroll
      for (int t = 0; t < 16; ++t) h[t] = __ldg(th + t);        // all hi-row reads in flight before any is used
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        const float4 l = tl[t];
        const uint64_t ch = f2_pack(h[t].x, h[t].y), sh = f2_pack(h[t].z, h[t].w), cl = f2_pack(l.x, l.y), sl = f2_pack(l.z, l.w);
        cs2[t] = f2_sub(f2_mul(ch, cl), f2_mul(sh, sl));
        sn2[t] = f2_fma(sh, cl, f2_mul(ch, sl));
      }
    };
    // The group's queries as the K-major, 128-byte-swizzled B operand: row 8 g + h, two 64-wide panels.  The
    // contraction runs over the dimensions in the order the epilogue leaves the rotated keys in: 16-byte piece
    // 8 hf + 2 c holds dimensions 32 hf + 8 c .. + 7, piece 8 hf + 2 c + 1 the dimensions 64 above them.
    // Only called when no score product that reads the rows can still be in flight.
    auto write_q = [&](int qs) {
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
        const int kc = ((ch & 7) >> 2) * 8 + (ch & 3) * 2 + (ch >> 3);     // position of the piece along the contraction
        const int qrow = (head / REP) * 8 + head % REP, c8 = kc & 7;
        *reinterpret_cast<uint4*>(sQ_ptr + (kc >> 3) * KT_Q_PANEL_BYTES + qrow * 128 + ((c8 ^ (qrow & 7)) << 4)) = val;
      }
      fence_proxy_async_smem();
    };
    // Scores of one slab: REP columns of its accumulator, scaled, rows past the tile's last token masked; the reading
    // half of the epilogue warps alternates from slab to slab.
    auto read_out = [&](const KtPending& p) -> bool {
      if (!(p.meta & KP_VALID) || (int)((p.meta >> 1) & 1u) != hf) return true;       // uniform over the warp
      const uint32_t sl_ = (p.meta >> 4) & 3u, par = (p.meta >> 6) & 1u, mode = (p.meta >> 2) & 3u;
      if (!__all_sync(0xffffffffu, mbar_wait(s_full + 8 * sl_, par, abort_flag))) return false;
      fence_after_sync();
      float sv[REP];
      {
        uint32_t* dst = reinterpret_cast<uint32_t*>(sv);
        const uint32_t src = lane_addr + TM_S + 16 * sl_;
        if constexpr (REP == 1) tmem_ld1(src, dst);
        else if constexpr (REP == 2) tmem_ld2(src, dst);
        else if constexpr (REP == 4) tmem_ld4(src, dst);
        else tmem_ld8(src, dst);
      }
      tmem_ld_wait();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty + 8 * sl_);
      const bool live = (p.meta & KP_LIVE) != 0;
      float* out = p.out;
#pragma unroll
      for (int i = 0; i < REP; ++i) {
        float x = sv[i] * sm_scale;
        if (mode == KP_ADD_FINAL) x += out[i];                                       // the first pass stored its part
        sv[i] = live ? x : -INFINITY;
      }
      if constexpr (REP >= 4) {
#pragma unroll
        for (int i = 0; i < REP; i += 4) *reinterpret_cast<float4*>(out + i) = make_float4(sv[i], sv[i + 1], sv[i + 2], sv[i + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < REP; ++i) out[i] = sv[i];
      }
      if (mode != KP_STORE_PART) {
        const int a_ = p.mxi;                                                        // slab index / 2: which maxima
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int i = 0; i < REP; ++i) tmax[a][i] = a == a_ ? fmaxf(tmax[a][i], sv[i]) : tmax[a][i];
      }
      return true;
    };
    // Folds this thread's running maxima into the per-(sequence, head) maximum: over the warp's rows first, then one
    // atomic per head (max is order-independent, so the result is deterministic).
    auto flush_max = [&](int qs) {
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int sli = 2 * a + hf;
        if (sli < Hkv) {
          const int g = sli + g_rot < Hkv ? sli + g_rot : sli + g_rot - Hkv;
          unsigned mine = 0u;
#pragma unroll
          for (int i = 0; i < REP; ++i) {
            const unsigned m = warp_max_u32(enc_ordered(tmax[a][i]));
            if (lane == i) mine = m;
            tmax[a][i] = -INFINITY;
          }
          if (lane < REP) atomicMax(&v.seqmax[qs * Hq + g * REP + lane], mine);
        }
      }
    };

    KtPending p_old{nullptr, 0, 0u}, p_new{nullptr, 0, 0u};
    int4 e = w0 < total ? klist[w0] : kt_none;
    if (w0 < total) { write_q(e.w); rope_setup(kpos[(size_t)e.x * TILE + row]); }
    for (int w = w0; w < total && ok; ++w) {
      const int4 nxt = w + 1 < total ? klist[w + 1] : kt_none;
      const int tile = e.x, cls = e.y & 0xff, n_valid = e.y >> 8, qs = e.w;
      const int passes = (cls + KT_A_SLOTS - 1) / KT_A_SLOTS;
      const int pos_next = nxt.w >= 0 ? kpos[(size_t)nxt.x * TILE + row] : 0;      // fetched now, used after the tile's slabs
      float* const out_row = v.scores + ((size_t)tile * TILE + row) * Hq;
      const uint32_t live_bit = row < n_valid ? KP_LIVE : 0u;
      for (int ps = 0; ps < passes && ok; ++ps) {
        const uint32_t mode = passes == 1 ? KP_STORE_FINAL : (ps == 0 ? KP_STORE_PART : KP_ADD_FINAL);
        for (int sli = 0; sli < Hkv; ++sli) {
          const int g = sli + g_rot < Hkv ? sli + g_rot : sli + g_rot - Hkv;
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(slab_full + 8 * sbuf, sph, abort_flag)))) break;
          fence_after_sync();
          const uint32_t sl_addr = lane_addr + TM_SLAB + sbuf * 128 + hf * 32;
          // the slab goes through the registers sixteen columns at a time (8 low dims + the 8 dims 64 above them), the
          // next piece's load in flight while this one is rotated; a piece's results overwrite the columns it came from
          uint32_t va[16], vb[16];
          tmem_ld8(sl_addr, va);
          tmem_ld8(sl_addr + 64, va + 8);
          if (!(ok = read_out(p_old))) break;                                // the scores of the slab before last
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t* cur = (c & 1) ? vb : va;
            uint32_t* nx = (c & 1) ? va : vb;
            tmem_ld_wait();
            if (c < 3) {
              tmem_ld8(sl_addr + 8 * (c + 1), nx);
              tmem_ld8(sl_addr + 64 + 8 * (c + 1), nx + 8);
            }
            // a rotated value leaves as two f16: the value with its low 13 mantissa bits cleared (exact in f16) and the
            // rest (rounded to f16: 2^-21 of the value instead of the 2^-11 of one f16), so that the score error stays
            // far below the bar even where a few key channels carry most of the magnitude
            uint32_t oh[8], ol[8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int t = 4 * c + u;
              const uint64_t L = f2_pack_bits(cur[2 * u], cur[2 * u + 1]), H = f2_pack_bits(cur[8 + 2 * u], cur[8 + 2 * u + 1]);
              const uint64_t a = f2_sub(f2_mul(L, cs2[t]), f2_mul(H, sn2[t]));           // lo cos - hi sin
              const uint64_t b = f2_fma(L, sn2[t], f2_mul(H, cs2[t]));                   // hi cos + lo sin
              const uint64_t ah = a & 0xFFFFE000FFFFE000ull, bh = b & 0xFFFFE000FFFFE000ull;
              oh[u] = f2_to_f16x2_sat(ah);
              oh[4 + u] = f2_to_f16x2_sat(bh);
              ol[u] = f2_to_f16x2_sat(f2_sub(a, ah));
              ol[4 + u] = f2_to_f16x2_sat(f2_sub(b, bh));
            }
            tmem_st8(sl_addr + 8 * c, oh);                                    // high parts: columns 0 .. 63 of the slab
            tmem_st8(sl_addr + 64 + 8 * c, ol);                               // low parts: columns 64 .. 127
          }
          tmem_st_wait();
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(kr_full + 8 * sbuf);
          p_old = p_new;
          p_new.out = out_row + g * REP;
          p_new.mxi = sli >> 1;
          p_new.meta = KP_VALID | ((uint32_t)(sli & 1) << 1) | (mode << 2) | (slot << 4) | (slph << 6) | live_bit;
          if (++sbuf == (uint32_t)KT_SLABS) { sbuf = 0; sph ^= 1u; }
          if (++slot == (uint32_t)KT_S_SLOTS) { slot = 0; slph ^= 1u; }
        }
      }
      if (!ok) break;
      if (nxt.w >= 0) rope_setup(pos_next);
      if (nxt.w != qs) {
        // last tile of this query slot in the piece: the owed read-outs belong to it; the query operand may only change
        // once every score product that reads the old one has retired
        if (!(ok = read_out(p_old))) break;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(s_full + 8 * ((p_new.meta >> 4) & 3u), (p_new.meta >> 6) & 1u, abort_flag)))) break;
        if (!(ok = read_out(p_new))) break;
        p_old.meta = 0u;
        p_new.meta = 0u;
        flush_max(qs);
        if (nxt.w >= 0) write_q(nxt.w);
      }
      e = nxt;
    }
    tmem_ld_wait();                                                          // nothing of this thread is in flight when TMEM is freed
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

// U_K^-1 [d x d] (row j = spectral component j) -> the B operand panels of the K-score kernel, each one contiguous:
// panel (j64, g) = rows n = 0..127 of 128 bytes, out[((j64 * Hkv + g) * 128 + n) * 64 + k] = in[(j64 * 64 + k) * d + g * 128 + n].
// A panel whose rows lie 2 d bytes apart (the plain transpose) sits in very few L2 slices, and with many CTAs asking
// for the same panel its copy took thousands of cycles; 16 KiB of consecutive lines spread over all of them.
// The first KT_HOT_PANELS panel rows (all that tiles of the narrow rank classes read) are stored KT_UINV_COPIES
// times, blockIdx.z selecting the copy: when every CTA of the K-score kernel works on narrow tiles they all ask L2
// for the same 8 .. 32 panels, and a panel's copy then took ~400 cycles per CTA asking for it (7 k cycles for a class-1
// tile's panel); with each CTA on one of eight copies the requests spread over eight times as many lines.
__global__ void uinv_panels_kernel(const unsigned short* __restrict__ in, unsigned short* __restrict__ out, int d) {
  __shared__ unsigned short t[64][129];
  const int j64 = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
  if (blockIdx.z > 0) {
    if (j64 >= KT_HOT_PANELS) return;
    out += (size_t)d * d + (size_t)(blockIdx.z - 1) * KT_HOT_PANELS * d * 64;
  }
  for (int i = tid; i < 64 * 128; i += blockDim.x) {
    const int k = i >> 7, n = i & 127;
    t[k][n] = in[(size_t)(j64 * 64 + k) * d + g * 128 + n];
  }
  __syncthreads();
  unsigned short* o = out + ((size_t)(j64 * gridDim.y + g) * 128) * 64;
  for (int i = tid; i < 64 * 128; i += blockDim.x) {
    const int n = i >> 6, k = i & 63;
    o[i] = t[k][n];
  }
}

cudaError_t launch_uinv_panels(const void* in, void* out, int d, cudaStream_t st) {
  ProfScope ps(TWKV_K_OTHER, st);
  uinv_panels_kernel<<<dim3(d / 64, d / 128, KT_UINV_COPIES), 256, 0, st>>>(reinterpret_cast<const unsigned short*>(in),
                                                           reinterpret_cast<unsigned short*>(out), d);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_transpose16(const void* in, void* out, int n, cudaStream_t st) {
  ProfScope ps(TWKV_K_OTHER, st);
  transpose16_kernel<<<dim3(n / 32, n / 32), dim3(32, 8), 0, st>>>(reinterpret_cast<const unsigned short*>(in),
                                                                    reinterpret_cast<unsigned short*>(out), n);
  count_launch();
  return cudaGetLastError();
}

// bytes of the re-tiled copy of one layer's U_K^-1 and the panel rows (of 128 x 64) it holds
size_t kscore_uinv_bytes(int d) { return (size_t)d * d * 2 + (size_t)(KT_UINV_COPIES - 1) * KT_HOT_PANELS * d * 64 * 2; }
size_t kscore_uinv_panel_rows(int d) { return (size_t)(d / 64) * d + (size_t)(KT_UINV_COPIES - 1) * KT_HOT_PANELS * d; }

size_t kscore_tc_smem_bytes(int nb) {
  return (size_t)(KT_A_SLOTS + nb) * PANEL_BYTES + 2 * KT_Q_PANEL_BYTES + KT_ROPE_STAGE_BYTES + 8 * (KT_N_BARS + 2 * nb) +
         2 * sizeof(int);
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
