// K-side of decode attention on the 5th-generation tensor cores.
//
// Per K tile (128 tokens of one rank class c, panels [128 x 64] in HBM) and per KV head g:
//   Kbar_g = X^_K[128 x 64c] . U_K^-1[0:64c, 128g : 128g+128]                 (Eq. 3)
//   Krot_g = RoPE(Kbar_g, position of each token)                             (keys are rotated after reconstruction)
//   S_g    = Krot_g . Q_g^T,  Q_g = the REP query heads that share KV head g   (the GQA group makes this a dense contraction)
// The first product is a tcgen05.mma chain (M = 128, N = 128, K = 16 per instruction) whose fp32
// accumulator lives in TMEM; X^_K panels and panels of the pre-transposed U_K^-1 arrive by TMA with
// the 128-byte swizzle, which is the K-major operand layout the MMA reads from shared memory.
// Epilogue warps pull the slab out of TMEM, rotate it in fp32, split it into a high and a low f16 part and
// store both back to TMEM, from where they are the A operands of the second product (N = 16, the group's
// heads padded; one product per part);
// its accumulator S stays in TMEM until the tile's last slab, so RoPE is the only per-element
// CUDA-core work.  Both sums are linear in X^_K, so a class wider than 8 panels runs as two passes
// over its panels that accumulate into the same S.
//
// Tensor memory (512 columns): slab accumulators 2 x 128 | rotated keys, high and low part, 64 each | S 8 x 16.
// Warp roles (384 threads, one persistent CTA per SM working through a contiguous, cost-balanced piece of the tile list):
//   warp 0      TMA producer of U_K^-1 panels (ring, one lane per stage)
//   warp 1      issuer of the main products (one elected lane; owns the TMEM allocation)
//   warps 2-9   epilogue (thread = one token row x one half of the RoPE frequencies)
//   warp 10     TMA producer of X^_K panels (ring of 8 slots served by four lanes, runs ahead into the next tile)
//   warp 11     issuer of the score products (one elected lane)
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
constexpr uint32_t KT_TMEM_COLS = 512;
constexpr uint32_t TM_SLAB = 0, TM_KR = 256, TM_S = 384;      // column offsets inside the allocation
constexpr uint32_t PANEL_BYTES = 16384;
constexpr int KT_Q_ROWS = 72;                                 // 8 rows per KV head + 8 rows of padding
constexpr uint32_t KT_Q_PANEL_BYTES = KT_Q_ROWS * 128;        // one 64-wide K panel of the query operand
constexpr int KT_ROPE_STRIDE = 65;                            // float2 per row of the small RoPE tables in shared memory (64 + 1 against bank conflicts)
constexpr uint32_t KT_ROPE_STAGE_BYTES = ROPE_SMALL_ROWS * KT_ROPE_STRIDE * 8;

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

template <bool BF16> __device__ __forceinline__ float kt_to_f32(unsigned short bits) {
  if constexpr (BF16) return __uint_as_float((unsigned)bits << 16);
  else return __half2float(__ushort_as_half(bits));
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
  float2* sRope = reinterpret_cast<float2*>(sQ_ptr + 2 * KT_Q_PANEL_BYTES);   // [32 rows][65]: the two small RoPE tables
  unsigned char* tail = sQ_ptr + 2 * KT_Q_PANEL_BYTES + KT_ROPE_STAGE_BYTES;
  const uint32_t bars = smem_addr(tail);
  // barrier map (8 bytes each)
  const uint32_t a_full = bars, a_empty = a_full + 8 * KT_A_SLOTS, b_full = a_empty + 8 * KT_A_SLOTS;
  const uint32_t b_empty = b_full + 8 * nb, slab_full = b_empty + 8 * nb, slab_empty = slab_full + 16;
  const uint32_t kr_full = slab_empty + 16, kr_empty = kr_full + 16, s_full = kr_empty + 16;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (2 * KT_A_SLOTS + 2 * nb + 9));
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
  if (warp == 1) tmem_alloc(smem_addr(s_tmem_base), KT_TMEM_COLS);
  for (int i = tid; i < 2 * (int)KT_Q_PANEL_BYTES / 16; i += KT_THREADS)        // padding rows of the query operand stay zero
    reinterpret_cast<uint4*>(sQ_ptr)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = tid; i < ROPE_SMALL_ROWS * 64; i += KT_THREADS) sRope[(i >> 6) * KT_ROPE_STRIDE + (i & 63)] = v.rope_lo[i];
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
  constexpr int wstep = 1;
  // CTAs walk the KV heads in rotated order, so that at any moment they read different panels of U_K^-1 from L2
  const int g_rot = blockIdx.x % Hkv;

  if (warp == 10) {
    // ------------------------------------------------------------- TMA producer: X^_K panels
    // A thread's TMA copies complete one after the other, so the ring is served by four lanes
    // (lane L owns slots L and L + 4) that each keep their own copy in flight.
    if (lane < 4) {
      if (lane == 0) tma_prefetch_desc(&map_blocks);
      uint32_t ak = 0;                                          // panels so far; slot = ak % 8
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; w += wstep) {
        const int4 nxt = w + wstep < total ? klist[w + wstep] : kt_none;
        const int cls = e.y & 0xff, blk = e.z;
        for (int j = 0; j < cls; ++j, ++ak) {
          const uint32_t slot = ak % KT_A_SLOTS, ph = (ak / KT_A_SLOTS) & 1u;
          if ((slot & 3u) != (uint32_t)lane) continue;
          if (!(ok = mbar_wait(a_empty + 8 * slot, ph ^ 1u, abort_flag))) break;
          mbar_expect_tx(a_full + 8 * slot, PANEL_BYTES);
          tma_load_2d(sA + slot * PANEL_BYTES, &map_blocks, a_full + 8 * slot, 0, (blk + j) * TILE);
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
    // one lane per ring stage, for the same reason
    if (lane < nb) {
      if (lane == 0) tma_prefetch_desc(&map_uinvT);
      uint32_t bk = 0, bst = 0, bph = 0;                        // panels so far; ring stage and its phase
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; w += wstep) {
        const int4 nxt = w + wstep < total ? klist[w + wstep] : kt_none;
        const int cls = e.y & 0xff;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const int np = min(KT_A_SLOTS, cls - p0);
          for (int sl = 0; sl < Hkv && ok; ++sl) {
            const int g = sl + g_rot < Hkv ? sl + g_rot : sl + g_rot - Hkv;
            for (int j = 0; j < np; ++j, ++bk) {
              const uint32_t st = bst, ph = bph;
              if (++bst == (uint32_t)nb) { bst = 0; bph ^= 1u; }
              if (st != (uint32_t)lane) continue;
              if (!(ok = mbar_wait(b_empty + 8 * st, ph ^ 1u, abort_flag))) break;
              mbar_expect_tx(b_full + 8 * st, PANEL_BYTES);
              tma_load_2d(sB + st * PANEL_BYTES, &map_uinvT, b_full + 8 * st, (p0 + j) * PANEL, g * HEAD_DIM);
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
      uint32_t bst = 0, bph = 0, ak = 0, sc = 0;
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; w += wstep) {
        const int4 nxt = w + wstep < total ? klist[w + wstep] : kt_none;
        const int cls = e.y & 0xff;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const int np = min(KT_A_SLOTS, cls - p0);
          for (int sl = 0; sl < Hkv && ok; ++sl) {
            const uint32_t buf = sc & 1u;
            if (!(ok = mbar_wait_thin(slab_empty + 8 * buf, ((sc >> 1) & 1u) ^ 1u, abort_flag))) break;
            const uint32_t d = tmem_base + TM_SLAB + buf * 128;
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
            mma_commit(slab_full + 8 * buf);                            // slab accumulator complete
            ++sc;
          }
          ak += np;
        }
        e = nxt;
      }
    }
    __syncwarp();
  } else if (warp == 11) {
    // ------------------------------------------------------------- score-product issuer (one elected lane)
    // S_g (+)= Krot_g . Q_g^T as soon as the epilogue warps have stored a rotated slab; a thread of its own, so that
    // neither issue stream waits for the other's barriers
    if (elect_one()) {
      const uint32_t idesc_s = idesc_f16(0, 128, 16);
      const uint32_t q_lo0 = kmajor_sw128_desc_lo(sQ);
      uint32_t sc = 0;
      bool ok = true;
      int4 e = w0 < total ? klist[w0] : kt_none;
      for (int w = w0; w < total && ok; w += wstep) {
        const int4 nxt = w + wstep < total ? klist[w + wstep] : kt_none;
        const int cls = e.y & 0xff;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const bool last_pass = p0 + KT_A_SLOTS >= cls;
          for (int sl = 0; sl < Hkv; ++sl, ++sc) {
            const int g = sl + g_rot < Hkv ? sl + g_rot : sl + g_rot - Hkv;
            if (!(ok = mbar_wait_thin(kr_full, sc & 1u, abort_flag))) break;
            fence_after_sync();
            // the rotated keys come as a high and a low f16 part (their sum carries 21 bits): two products into the same S
            mma_f16_ts_k128(tmem_base + TM_S + 16 * g, tmem_base + TM_KR, q_lo0 + g * (1024 >> 4), KT_Q_PANEL_BYTES >> 4, idesc_s,
                            p0 > 0 ? 1u : 0u);
            mma_f16_ts_k128(tmem_base + TM_S + 16 * g, tmem_base + TM_KR + 64, q_lo0 + g * (1024 >> 4), KT_Q_PANEL_BYTES >> 4, idesc_s, 1u);
            mma_commit(kr_empty);
            if (last_pass && sl == Hkv - 1) mma_commit(s_full);        // the tile's scores are complete
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
    const int g_lo = hf ? (Hkv + 1) / 2 : 0, g_hi = hf ? Hkv : (Hkv + 1) / 2;      // this thread's KV-head groups (at most 4)
    const float sm_scale = v.sm_scale;
    const int* kpos = v.aux(layer, 0);
    const float2* __restrict__ rope_hi = v.rope_hi;
    uint32_t sc = 0, tcount = 0;
    bool ok = true, slab_ready = false;                            // slab_ready: the next slab's accumulator was already seen complete
    float cs[32], sn[32];                                         // scratch of rope_setup
    uint64_t cs2[16], sn2[16];                                    // the tile's rotation factors, frequencies (2 t, 2 t + 1) packed
    float tmax[4 * REP];                                            // running maxima of this thread's heads for the current query slot
#pragma unroll
    for (int i = 0; i < 4 * REP; ++i) tmax[i] = -INFINITY;

    // cos / sin of (row, frequency): pos = hi * 256 + mid * 16 + lo, the three table rows combine by the angle-addition
    // formulas.  The mid and lo rows come from shared memory (padded rows: lanes with different rows hit different
    // banks), the hi row from global memory: a tile's 128 rows share a few hi rows, so those reads stay in L1.
    auto rope_setup = [&](int pos) {
      const float2* __restrict__ th = rope_hi + (size_t)((pos >> 8) & (ROPE_HI - 1)) * 64 + hf * 32;
      const float2* tm = sRope + ((pos >> 4) & 15) * KT_ROPE_STRIDE + hf * 32;
      const float2* tl = sRope + (16 + (pos & 15)) * KT_ROPE_STRIDE + hf * 32;
#pragma unroll
      for (int t = 0; t < 32; t += 2) {                        // all hi-row reads in flight before any is used
        const float4 h = __ldg(reinterpret_cast<const float4*>(th + t));
        cs[t] = h.x; sn[t] = h.y; cs[t + 1] = h.z; sn[t + 1] = h.w;
      }
#pragma unroll
      for (int t = 0; t < 32; ++t) {
        const float2 m = tm[t], l = tl[t];
        const float hx = cs[t] * m.x - sn[t] * m.y, hy = sn[t] * m.x + cs[t] * m.y;
        cs[t] = hx * l.x - hy * l.y;
        sn[t] = hy * l.x + hx * l.y;
      }
#pragma unroll
      for (int t = 0; t < 16; ++t) { cs2[t] = f2_pack(cs[2 * t], cs[2 * t + 1]); sn2[t] = f2_pack(sn[2 * t], sn[2 * t + 1]); }
    };
    // The group's queries as the K-major, 128-byte-swizzled B operand: row 8 g + h, two 64-wide panels.
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
        const int qrow = (head / REP) * 8 + head % REP, c8 = ch & 7;
        *reinterpret_cast<uint4*>(sQ_ptr + (ch >> 3) * KT_Q_PANEL_BYTES + qrow * 128 + ((c8 ^ (qrow & 7)) << 4)) = val;
      }
      fence_proxy_async_smem();
    };

    int4 e = w0 < total ? klist[w0] : kt_none;
    if (w0 < total) { write_q(e.w); rope_setup(kpos[(size_t)e.x * TILE + row]); }
    for (int w = w0; w < total && ok; w += wstep) {
      const int4 nxt = w + wstep < total ? klist[w + wstep] : kt_none;
      const int tile = e.x, cls = e.y & 0xff, n_valid = e.y >> 8, qs = e.w;
      const int n_slabs = ((cls + KT_A_SLOTS - 1) / KT_A_SLOTS) * Hkv;
      const int pos_next = nxt.w >= 0 ? kpos[(size_t)nxt.x * TILE + row] : 0;      // fetched now, used after the tile's slabs
      for (int sl = 0; sl < n_slabs; ++sl, ++sc) {
        const uint32_t buf = sc & 1u, par = (sc >> 1) & 1u;
        // barrier probes cost a few hundred cycles of latency each, so each is issued early (the next slab's "full"
        // during this slab's store, "rotated keys free" before the rotation) and only waited on if it had not flipped yet
        if (!slab_ready && !(ok = __all_sync(0xffffffffu, mbar_wait(slab_full + 8 * buf, par, abort_flag)))) break;
        fence_after_sync();
        const uint32_t slab = lane_addr + TM_SLAB + buf * 128 + hf * 32;
        const uint32_t kr = lane_addr + TM_KR + hf * 16;                     // high parts; the low parts 64 columns on
        const uint32_t kr_par = (sc & 1u) ^ 1u;
        uint32_t lo[32], hi[32];
        tmem_ld32(slab, lo);
        tmem_ld32(slab + 64, hi);
        const bool kr_probe = mbar_try(kr_empty, kr_par);
        tmem_ld_wait();
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(slab_empty + 8 * buf);                    // the slab accumulator is free for slab n + 2
        // a rotated value v leaves as two f16: v with its low 13 mantissa bits cleared (exact in f16) and the rest
        // (rounded to f16: 2^-21 of v instead of the 2^-11 of one f16), so that the score error stays far below the bar
        // even where a few key channels carry most of the magnitude
#pragma unroll
        for (int hb = 0; hb < 2; ++hb) {
          uint32_t p1[8], p2[8], l1[8], l2[8];
#pragma unroll
          for (int t8 = 0; t8 < 8; ++t8) {
            const int t = hb * 8 + t8;
            const uint64_t L = f2_pack_bits(lo[2 * t], lo[2 * t + 1]), H = f2_pack_bits(hi[2 * t], hi[2 * t + 1]);
            const uint64_t a = f2_sub(f2_mul(L, cs2[t]), f2_mul(H, sn2[t]));           // lo cos - hi sin
            const uint64_t b = f2_fma(L, sn2[t], f2_mul(H, cs2[t]));                   // hi cos + lo sin
            const uint64_t ah = a & 0xFFFFE000FFFFE000ull, bh = b & 0xFFFFE000FFFFE000ull;
            p1[t8] = f2_to_f16x2_sat(ah);
            p2[t8] = f2_to_f16x2_sat(bh);
            l1[t8] = f2_to_f16x2_sat(f2_sub(a, ah));
            l2[t8] = f2_to_f16x2_sat(f2_sub(b, bh));
          }
          if (hb == 0) {
            if (!__all_sync(0xffffffffu, kr_probe) && !(ok = __all_sync(0xffffffffu, mbar_wait(kr_empty, kr_par, abort_flag)))) break;
            fence_after_sync();
          }
          tmem_st8(kr + 8 * hb, p1);                                        // dims d -> column d / 2
          tmem_st8(kr + 32 + 8 * hb, p2);                                   // dims 64 + d
          tmem_st8(kr + 64 + 8 * hb, l1);
          tmem_st8(kr + 96 + 8 * hb, l2);
        }
        if (!ok) break;
        const bool next_probe = mbar_try(slab_full + 8 * (buf ^ 1u), ((sc + 1) >> 1) & 1u);
        tmem_st_wait();
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(kr_full);
        slab_ready = __all_sync(0xffffffffu, next_probe);
      }
      if (!ok) break;
      // the next tile's rotation factors are fetched while this tile's last score products drain
      if (nxt.w >= 0) rope_setup(pos_next);
      // all score products of the tile have retired: scale, mask the rows past the last token, store
      if (!(ok = __all_sync(0xffffffffu, mbar_wait(s_full, tcount & 1u, abort_flag)))) break;
      ++tcount;
      fence_after_sync();
      {
        // this thread's groups g_lo .. g_hi - 1: REP columns of each group's 16-column region, all loads in flight at once
        float sv[4 * REP];
#pragma unroll
        for (int gi = 0; gi < 4; ++gi)
          if (g_lo + gi < g_hi) {
            uint32_t* dst = reinterpret_cast<uint32_t*>(sv + gi * REP);
            const uint32_t src = lane_addr + TM_S + 16 * (g_lo + gi);
            if constexpr (REP == 1) tmem_ld1(src, dst);
            else if constexpr (REP == 2) tmem_ld2(src, dst);
            else if constexpr (REP == 4) tmem_ld4(src, dst);
            else tmem_ld8(src, dst);
          }
        tmem_ld_wait();
        const int h0 = g_lo * REP, nh = (g_hi - g_lo) * REP;
        float* out = v.scores + ((size_t)tile * TILE + row) * Hq + h0;
        const bool live = row < n_valid;
#pragma unroll
        for (int i = 0; i < 4 * REP; ++i) sv[i] = (live && i < nh) ? sv[i] * sm_scale : -INFINITY;
        if constexpr (REP >= 4) {
#pragma unroll
          for (int i = 0; i < 4 * REP; i += 4)
            if (i < nh) *reinterpret_cast<float4*>(out + i) = make_float4(sv[i], sv[i + 1], sv[i + 2], sv[i + 3]);
        } else {
#pragma unroll
          for (int i = 0; i < 4 * REP; ++i) if (i < nh) out[i] = sv[i];
        }
#pragma unroll
        for (int i = 0; i < 4 * REP; ++i) tmax[i] = fmaxf(tmax[i], sv[i]);
        if (nxt.w != qs) {
          // last tile of this query slot in the piece: maximum over the warp's rows, one atomic per head
#pragma unroll
          for (int i = 0; i < 4 * REP; ++i) {
            float m = tmax[i];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (lane == i && i < nh) atomicMax(&v.seqmax[qs * Hq + h0 + i], enc_ordered(m));
            tmax[i] = -INFINITY;
          }
        }
      }
      if (nxt.w >= 0 && nxt.w != qs) write_q(nxt.w);
      e = nxt;
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
  return (size_t)(KT_A_SLOTS + nb) * PANEL_BYTES + 2 * KT_Q_PANEL_BYTES + KT_ROPE_STAGE_BYTES + 8 * (2 * KT_A_SLOTS + 2 * nb + 9) +
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
