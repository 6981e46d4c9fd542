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
// Each slab's scores land in one of four 16-column accumulators and are read out by four warps of their own (scaled,
// masked, stored, folded into the per-(sequence, head) maximum), so that the rotating warps never wait for a score
// product and a tile has no tail: RoPE and the high / low split are the only per-element CUDA-core work.  Both products
// are linear in X^_K, so a class wider than 8 panels runs as two passes over its panels; the second pass adds to the
// scores the first one stored.
//
// Tensor memory (512 columns): slabs 3 x 128 | score accumulators 4 x 16.
// Warp roles (512 threads, one persistent CTA per SM working through a contiguous, cost-balanced piece of the tile list;
// the register file is re-divided by warpgroup with setmaxnreg: 56 registers per thread for the light roles, 184 for the
// rotating warps, which then hold a slab's registers without spilling):
//   warp 0      TMA producer of U_K^-1 panels (ring; one elected lane)
//   warp 1      issuer of the main products (one elected lane; owns the TMEM allocation)
//   warp 2      TMA producer of X^_K panels (ring of 8 slots; one elected lane, runs ahead into the next tiles)
//   warp 3      issuer of the score products (one elected lane)
//   warps 4-11  epilogue (thread = one token row x one half of the RoPE frequencies): rotation, high / low split
//   warps 12-15 score read-out (thread = one token row)
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

constexpr int KT_THREADS = 512;
constexpr int KT_EPI = 256;
constexpr int KT_REGS_LIGHT = 56, KT_REGS_EPI = 184;         // registers per thread after the roles re-divide the register file
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

__device__ __forceinline__ void regs_shrink() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(KT_REGS_LIGHT)); }
__device__ __forceinline__ void regs_grow() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(KT_REGS_EPI)); }

template <bool BF16> __device__ __forceinline__ float kt_to_f32(unsigned short bits) {
  if constexpr (BF16) return __uint_as_float((unsigned)bits << 16);
  else return __half2float(__ushort_as_half(bits));
}

constexpr uint32_t KP_STORE_PART = 0u, KP_STORE_FINAL = 1u, KP_ADD_FINAL = 2u, KP_DISCARD = 3u;      // what a read-out does with a slab's scores
constexpr int KE_DISCARD = 0x80;                               // list entry, .y bit 7: a filler tile whose scores are not kept

// PAIR: the kernel runs on CTA pairs (clusters of two, cta_group::2).  The two CTAs take two tiles of the same class
// at a time: each loads its own tile's panels and its own 64 of the 128 rows of every U_K^-1 panel, one
// tcgen05.mma of the even CTA (M = 256 over the pair) drives both tensor cores, each CTA's accumulator in its own
// TMEM.  Per SM the panels of U_K^-1 read from L2, and the shared-memory operand reads, drop by half; both bound the
// single-CTA kernel on the wide classes.  Epilogue, rotation factors and queries stay per CTA; the score product
// takes 8 query rows from each CTA (N = 16), so each CTA finds its own scores in its own 8 columns.
// Barriers: a_full / b_full / kr_full / slab_empty / s_empty live in the even CTA (the odd CTA's copies complete on
// them and its epilogue warps arrive on them through the cluster window); a_empty / b_empty / slab_full / s_full exist in
// both and are signalled together by a multicast tcgen05.commit (a commit, not a load).
// DBG (caches created with TWKV_DEBUG=1): rotated keys that the f16 conversion clamps are reported.
template <bool BF16, int REP, bool PAIR, bool DBG>
__global__ void __launch_bounds__(KT_THREADS, 1)
kscore_tc_kernel(const __grid_constant__ CUtensorMap map_blocks, const __grid_constant__ CUtensorMap map_uinvT,
                 DevView v, int layer, const unsigned short* __restrict__ q, int nb) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  constexpr int CG = PAIR ? 2 : 1;
  // a ring stage of U_K^-1 holds two consecutive panels of one KV head (their halves in a pair CTA): one barrier wait
  // and one commit per eight MMAs keeps the issuing thread's own instructions below the tensor pipe's time
  constexpr uint32_t B_PART_BYTES = PAIR ? PANEL_BYTES / 2 : PANEL_BYTES;
  constexpr uint32_t B_STAGE_BYTES = 2 * B_PART_BYTES;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hq = v.Hq, Hkv = v.Hkv;
  const uint32_t crank = PAIR ? cluster_cta_rank() : 0u;
  // operand tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t sA = smem_addr(smem_raw);
  const bool misaligned = (sA & 1023u) != 0;
  const uint32_t sB = sA + KT_A_SLOTS * PANEL_BYTES;
  const uint32_t sQ = sB + nb * B_STAGE_BYTES;
  unsigned char* sQ_ptr = smem_raw + KT_A_SLOTS * PANEL_BYTES + nb * B_STAGE_BYTES;
  float4* sRope = reinterpret_cast<float4*>(sQ_ptr + 2 * KT_Q_PANEL_BYTES);   // [16 rows][33]: the small RoPE table
  unsigned char* tail = sQ_ptr + 2 * KT_Q_PANEL_BYTES + KT_ROPE_STAGE_BYTES;
  const uint32_t bars = smem_addr(tail);
  // barrier map (8 bytes each)
  const uint32_t a_full = bars, a_empty = a_full + 8 * KT_A_SLOTS, b_full = a_empty + 8 * KT_A_SLOTS;
  const uint32_t b_empty = b_full + 8 * nb, slab_full = b_empty + 8 * nb, kr_full = slab_full + 8 * KT_SLABS;
  const uint32_t slab_empty = kr_full + 8 * KT_SLABS, s_full = slab_empty + 8 * KT_SLABS, s_empty = s_full + 8 * KT_S_SLOTS;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (KT_N_BARS + 2 * nb));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);
  // the even CTA's copies of the barriers both CTAs signal
  const uint32_t a_full_own = PAIR ? cluster_map(a_full, 0) : a_full, b_full_own = PAIR ? cluster_map(b_full, 0) : b_full;
  const uint32_t kr_full_own = PAIR ? cluster_map(kr_full, 0) : kr_full, s_empty_own = PAIR ? cluster_map(s_empty, 0) : s_empty;

  if (tid == 0) {
    for (int i = 0; i < KT_A_SLOTS; ++i) { mbar_init(a_full + 8 * i, 1); mbar_init(a_empty + 8 * i, 1); }
    for (int i = 0; i < nb; ++i) { mbar_init(b_full + 8 * i, 1); mbar_init(b_empty + 8 * i, 1); }
    for (int i = 0; i < KT_SLABS; ++i) {
      mbar_init(slab_full + 8 * i, 1); mbar_init(kr_full + 8 * i, CG * (KT_EPI / 32)); mbar_init(slab_empty + 8 * i, 1);
    }
    for (int i = 0; i < KT_S_SLOTS; ++i) { mbar_init(s_full + 8 * i, 1); mbar_init(s_empty + 8 * i, CG * 4); }
    *abort_flag = misaligned ? 1 : 0;
    mbar_init_fence();
  }
  if (warp == 1) {
    if constexpr (PAIR) tmem_alloc_pair(smem_addr(s_tmem_base), KT_TMEM_COLS);
    else tmem_alloc(smem_addr(s_tmem_base), KT_TMEM_COLS);
  }
  for (int i = tid; i < 2 * (int)KT_Q_PANEL_BYTES / 16; i += KT_THREADS)        // padding rows of the query operand stay zero
    reinterpret_cast<uint4*>(sQ_ptr)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = tid; i < ROPE_LO * 32; i += KT_THREADS) sRope[(i >> 5) * KT_ROPE_STRIDE + (i & 31)] = v.rope_lo[i];
  fence_proxy_async_smem();
  fence_before_sync();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();                       // both CTAs' barriers and TMEM are ready
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // Work list written by plan_kernel: the K tiles of the sequences being decoded, widest class first; this CTA's (this
  // pair's) contiguous piece [w0, total) of it, cut by estimated cost.  The pair list holds two entries per item, the
  // even CTA's and the odd CTA's tile, always of one class (a class with an odd number of tiles ends with a filler).
  const int piece = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int w0 = v.cta_start[piece], total = v.cta_start[piece + 1];
  const int4* klist = PAIR ? v.kpairs + crank : v.klist;
  constexpr int KSTEP = PAIR ? 2 : 1;
  const int4 kt_none = make_int4(0, 0, 0, -1);
  // CTAs walk the KV heads in rotated order, so that at any moment they read different panels of U_K^-1 from L2
  const int g_rot = piece % Hkv;

  if (misaligned) {
    // nothing was started; fall through to the common exit
  } else if (warp < 4) {
    regs_shrink();                                              // the register file is re-divided by role, whole warpgroups at a time
    if (warp == 2) {
    // ------------------------------------------------------------- TMA producer: X^_K panels
    // One elected thread issues every copy, in ring order (slots free up in that order, so waiting for the oldest one
    // never holds back a copy that could go out), and runs ahead into the next tiles.  Only a thread picked by
    // elect.sync issues the copy instruction directly; from lanes picked by their index each issue took hundreds of cycles.
    if (elect_one()) {
      tma_prefetch_desc(&map_blocks);
      uint32_t ak = 0;                                          // panels so far; slot = ak % 8
      bool ok = true;
      int4 e = w0 < total ? klist[KSTEP * w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[KSTEP * (w + 1)] : kt_none;
        const int cls = e.y & 0x7f, blk = e.z;
        for (int j = 0; j < cls; ++j, ++ak) {
          const uint32_t slot = ak % KT_A_SLOTS, ph = (ak / KT_A_SLOTS) & 1u;
          if (!(ok = mbar_wait_thin(a_empty + 8 * slot, ph ^ 1u, abort_flag))) break;
          if (crank == 0) mbar_expect_tx(a_full + 8 * slot, CG * PANEL_BYTES);          // this CTA's copy and the partner's
          if constexpr (PAIR) tma_load_2d_pair(sA + slot * PANEL_BYTES, &map_blocks, a_full_own + 8 * slot, 0, (blk + j) * TILE);
          else tma_load_2d(sA + slot * PANEL_BYTES, &map_blocks, a_full + 8 * slot, 0, (blk + j) * TILE);
        }
        e = nxt;
      }
      if (!ok && !PAIR)                                         // let copies in flight land before the CTA goes away
        for (uint32_t i = 0; i < (uint32_t)KT_A_SLOTS && i < ak; ++i) {
          const uint32_t n = ak - 1 - i;
          mbar_wait_drain(a_full + 8 * (n % KT_A_SLOTS), (n / KT_A_SLOTS) & 1u);
        }
    }
    __syncwarp();
  } else if (warp == 0) {
    // ------------------------------------------------------------- TMA producer: U_K^-1 panels
    // one elected thread, ring order, as above; a pair CTA loads its own half of every panel's rows
    if (elect_one()) {
      tma_prefetch_desc(&map_uinvT);
      uint32_t bk = 0, bst = 0, bph = 0;                        // panels so far; ring stage and its phase
      bool ok = true;
      int4 e = w0 < total ? klist[KSTEP * w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[KSTEP * (w + 1)] : kt_none;
        const int cls = e.y & 0x7f;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const int np = min(KT_A_SLOTS, cls - p0);
          for (int sl = 0; sl < Hkv && ok; ++sl) {
            const int g = sl + g_rot < Hkv ? sl + g_rot : sl + g_rot - Hkv;
            for (int j = 0; j < np; j += 2, ++bk) {
              const uint32_t st = bst, ph = bph;
              if (++bst == (uint32_t)nb) { bst = 0; bph ^= 1u; }
              if (!(ok = mbar_wait_thin(b_empty + 8 * st, ph ^ 1u, abort_flag))) break;
              const int npan = min(2, np - j);
              if (crank == 0) mbar_expect_tx(b_full + 8 * st, CG * npan * B_PART_BYTES);
              for (int k = 0; k < npan; ++k) {
                const int y = ((p0 + j + k) * Hkv + g) * HEAD_DIM + (PAIR ? (int)crank * (HEAD_DIM / 2) : 0);     // rows of the re-tiled copy
                if constexpr (PAIR) tma_load_2d_pair(sB + st * B_STAGE_BYTES + k * B_PART_BYTES, &map_uinvT, b_full_own + 8 * st, 0, y);
                else tma_load_2d(sB + st * B_STAGE_BYTES + k * B_PART_BYTES, &map_uinvT, b_full + 8 * st, 0, y);
              }
            }
          }
        }
        e = nxt;
      }
      if (!ok && !PAIR)
        for (uint32_t i = 0; i < (uint32_t)nb && i < bk; ++i) {
          const uint32_t n = bk - 1 - i;
          mbar_wait_drain(b_full + 8 * (n % nb), (n / nb) & 1u);
        }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (one elected lane runs the whole role)
    if (crank == 0 && elect_one()) {
      // This role is one thread issuing asynchronous work; what it costs is its own instruction stream (a 64-cycle MMA
      // per few instructions), so descriptors are stepped with 32-bit adds, a panel's four MMAs are one asm block, and
      // every wait tries once inline before it falls into the bounded loop.
      const uint32_t idesc_main = idesc_f16(BF16 ? 1 : 0, PAIR ? 256 : 128, 128);
      const uint32_t a_lo0 = kmajor_sw128_desc_lo(sA), b_lo0 = kmajor_sw128_desc_lo(sB);
      uint32_t bst = 0, bph = 0, ak = 0, sbuf = 0, sph = 0;
      bool ok = true;
      int4 e = w0 < total ? klist[KSTEP * w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[KSTEP * (w + 1)] : kt_none;
        const int cls = e.y & 0x7f;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          const int np = min(KT_A_SLOTS, cls - p0);
          for (int sl = 0; sl < Hkv && ok; ++sl) {
            // the buffer is free once the score products over its previous contents have retired
            if (!(ok = mbar_wait_thin(slab_empty + 8 * sbuf, sph ^ 1u, abort_flag))) break;
            fence_after_sync();
            const uint32_t d = tmem_base + TM_SLAB + sbuf * 128;
            const bool first = sl == 0, last = sl == Hkv - 1;
            uint32_t an = ak;
            for (int j = 0; j < np; j += 2, an += 2) {
              const bool two = j + 1 < np;
              const uint32_t slot = an & (KT_A_SLOTS - 1), slot2 = (an + 1) & (KT_A_SLOTS - 1);
              if (first) {
                if (!(ok = mbar_wait_thin(a_full + 8 * slot, (an >> 3) & 1u, abort_flag))) break;
                if (two && !(ok = mbar_wait_thin(a_full + 8 * slot2, ((an + 1) >> 3) & 1u, abort_flag))) break;
              }
              const uint32_t st = bst;
              if (!(ok = mbar_wait_thin(b_full + 8 * st, bph, abort_flag))) break;
              if (++bst == (uint32_t)nb) { bst = 0; bph ^= 1u; }
              fence_after_sync();
              mma_f16_ss_panel_cg<CG>(d, a_lo0 + slot * (PANEL_BYTES >> 4), b_lo0 + st * (B_STAGE_BYTES >> 4), idesc_main, j > 0 ? 1u : 0u);
              if (two) mma_f16_ss_panel_cg<CG>(d, a_lo0 + slot2 * (PANEL_BYTES >> 4), b_lo0 + st * (B_STAGE_BYTES >> 4) + (B_PART_BYTES >> 4), idesc_main, 1u);
              // ring stage reusable when these MMAs retire; after the last slab of the pass the X^_K panels are done too
              if constexpr (PAIR) {
                mma_commit_pair_both(b_empty + 8 * st);
                if (last) { mma_commit_pair_both(a_empty + 8 * slot); if (two) mma_commit_pair_both(a_empty + 8 * slot2); }
              } else {
                mma_commit(b_empty + 8 * st);
                if (last) { mma_commit(a_empty + 8 * slot); if (two) mma_commit(a_empty + 8 * slot2); }
              }
            }
            if (!ok) break;
            if constexpr (PAIR) mma_commit_pair_both(slab_full + 8 * sbuf);     // slab accumulator complete
            else mma_commit(slab_full + 8 * sbuf);
            if (++sbuf == (uint32_t)KT_SLABS) { sbuf = 0; sph ^= 1u; }
          }
          ak += np;
        }
        e = nxt;
      }
    }
    __syncwarp();
  } else if (warp == 3) {
    // ------------------------------------------------------------- score-product issuer (one elected lane)
    // S (+)= Krot_g . Q_g^T as soon as the epilogue warps have stored a rotated slab; a thread of its own, so that
    // neither issue stream waits for the other's barriers
    if (crank == 0 && elect_one()) {
      const uint32_t idesc_s = idesc_f16(0, PAIR ? 256 : 128, 16);
      const uint32_t q_lo0 = kmajor_sw128_desc_lo(sQ);
      uint32_t sbuf = 0, sph = 0, slot = 0, slph = 0;
      bool ok = true;
      int4 e = w0 < total ? klist[KSTEP * w0] : kt_none;
      for (int w = w0; w < total && ok; ++w) {
        const int4 nxt = w + 1 < total ? klist[KSTEP * (w + 1)] : kt_none;
        const int cls = e.y & 0x7f;
        for (int p0 = 0; p0 < cls && ok; p0 += KT_A_SLOTS) {
          for (int sl = 0; sl < Hkv; ++sl) {
            const int g = sl + g_rot < Hkv ? sl + g_rot : sl + g_rot - Hkv;
            if (!(ok = mbar_wait_thin(kr_full + 8 * sbuf, sph, abort_flag))) break;
            if (!(ok = mbar_wait_thin(s_empty + 8 * slot, slph ^ 1u, abort_flag))) break;
            fence_after_sync();
            // the rotated keys come as a high and a low f16 part (their sum carries 21 bits): two products into the same S
            const uint32_t kr = tmem_base + TM_SLAB + sbuf * 128, sd = tmem_base + TM_S + 16 * slot;
            mma_f16_ts_k128_cg<CG>(sd, kr, q_lo0 + g * (1024 >> 4), KT_Q_PANEL_BYTES >> 4, idesc_s, 0u);
            mma_f16_ts_k128_cg<CG>(sd, kr + 64, q_lo0 + g * (1024 >> 4), KT_Q_PANEL_BYTES >> 4, idesc_s, 1u);
            if constexpr (PAIR) { mma_commit_pair(slab_empty + 8 * sbuf); mma_commit_pair_both(s_full + 8 * slot); }
            else { mma_commit(slab_empty + 8 * sbuf); mma_commit(s_full + 8 * slot); }   // buffer reusable; scores complete
            if (++sbuf == (uint32_t)KT_SLABS) { sbuf = 0; sph ^= 1u; }
            if (++slot == (uint32_t)KT_S_SLOTS) { slot = 0; slph ^= 1u; }
          }
        }
        e = nxt;
      }
    }
    __syncwarp();
    }
  } else if (warp >= 4 && warp <= 11) {
    regs_grow();                                                // the rotating warps take what the light roles gave up
    // ------------------------------------------------------------- epilogue
    const int et = tid - 128;
    const int quarter = warp & 3, hf = (warp - 4) >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int* kpos = v.aux(layer, 0);
    const float4* __restrict__ rope_hi = v.rope_hi;
    uint32_t sbuf = 0, sph = 0, slot = 0, slph = 0;
    bool ok = true;
    uint64_t cs2[16], sn2[16];                                    // the tile's rotation factors, frequencies (2 t, 2 t + 1) packed
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
      const int qrow_of = v.qmap ? v.qmap[qs] : qs;                        // the row of q this query slot stands for
      for (int i = et; i < Hq * 16; i += KT_EPI) {
        const int head = i >> 4, ch = i & 15;                               // 8 dims per chunk
        const uint4 raw = *reinterpret_cast<const uint4*>(q + ((size_t)qrow_of * Hq + head) * HEAD_DIM + ch * 8);
        uint4 val = raw;
        if constexpr (BF16) {
          const unsigned short* e = reinterpret_cast<const unsigned short*>(&raw);
          // a bf16 query enters the score product as f16: one beyond the f16 range would be clamped, so it is reported
          bool over = false;
#pragma unroll
          for (int k = 0; k < 8; ++k) over |= !(fabsf(kt_to_f32<true>(e[k])) <= 65504.f);
          if (over) set_status(v, TWKV_ERR_DEVICE_CHECK);
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
    uint32_t last_slot = 0, last_slph = 0;                          // score accumulator of the slab rotated last, and its phase
    int4 e = w0 < total ? klist[KSTEP * w0] : kt_none;
    int pos_cur = w0 < total ? kpos[(size_t)e.x * TILE + row] : 0;              // this row's position in the current tile
    if (w0 < total) { write_q(e.w); rope_setup(pos_cur); }
    for (int w = w0; w < total && ok; ++w) {
      const int4 nxt = w + 1 < total ? klist[KSTEP * (w + 1)] : kt_none;
      const int cls = e.y & 0x7f, qs = e.w;
      [[maybe_unused]] const int n_valid = e.y >> 8;
      const int passes = (cls + KT_A_SLOTS - 1) / KT_A_SLOTS;
      const int pos_next = nxt.w >= 0 ? kpos[(size_t)nxt.x * TILE + row] : 0;      // fetched now, used after the tile's slabs
      for (int ps = 0; ps < passes && ok; ++ps) {
        for (int sli = 0; sli < Hkv; ++sli) {
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(slab_full + 8 * sbuf, sph, abort_flag)))) break;
          fence_after_sync();
          const uint32_t sl_addr = lane_addr + TM_SLAB + sbuf * 128 + hf * 32;
          // the slab goes through the registers sixteen columns at a time (8 low dims + the 8 dims 64 above them), the
          // next piece's load in flight while this one is rotated; a piece's results overwrite the columns it came from
          uint32_t va[16], vb[16];
          tmem_ld8(sl_addr, va);
          tmem_ld8(sl_addr + 64, va + 8);
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
            if constexpr (DBG) {
              // TWKV_DEBUG: a rotated key beyond the f16 range was clamped by the conversion above (its high part reads
              // 0x7bff); without the flag that goes unreported
              bool sat = false;
#pragma unroll
              for (int u = 0; u < 8; ++u) sat |= (oh[u] & 0x7fffu) == 0x7bffu || ((oh[u] >> 16) & 0x7fffu) == 0x7bffu;
              if (sat && row < n_valid) set_status(v, TWKV_ERR_DEVICE_CHECK);
            }
            tmem_st8(sl_addr + 8 * c, oh);                                    // high parts: columns 0 .. 63 of the slab
            tmem_st8(sl_addr + 64 + 8 * c, ol);                               // low parts: columns 64 .. 127
          }
          tmem_st_wait();
          fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(kr_full_own + 8 * sbuf);
            else mbar_arrive(kr_full + 8 * sbuf);
          }
          last_slot = slot; last_slph = slph;
          if (++sbuf == (uint32_t)KT_SLABS) { sbuf = 0; sph ^= 1u; }
          if (++slot == (uint32_t)KT_S_SLOTS) { slot = 0; slph ^= 1u; }
        }
      }
      if (!ok) break;
      if (nxt.w >= 0) rope_setup(pos_next);
      pos_cur = pos_next;
      if (nxt.w != qs) {
        // last tile of this query slot in the piece: the query operand may only change once every score product that
        // reads the old one has retired; they retire in order, and the last pair completes the accumulator of the slab rotated last
        if (nxt.w >= 0) {
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(s_full + 8 * last_slot, last_slph, abort_flag)))) break;
          write_q(nxt.w);
        }
      }
      e = nxt;
    }
    tmem_ld_wait();                                                          // nothing of this thread is in flight when TMEM is freed
  } else if (warp >= 12) {
    regs_shrink();
    // ------------------------------------------------------------- score read-out
    // One warp per TMEM lane quarter (thread = token row) follows the score issuer: REP columns of a slab's accumulator
    // as soon as its two products have retired, scaled, rows past the tile's last token (and, for a causal query, tokens
    // after it) masked, stored, and folded into the per-(sequence, head) maximum (over the warp's rows first, then one
    // atomic per head; max is order-independent, so the result is deterministic).  The rotating warps never wait for it.
    const int quarter = warp & 3, row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_col0 = TM_S + (PAIR ? 8u * crank : 0u);     // this CTA's columns of a score accumulator
    const float sm_scale = v.sm_scale;
    const int* kpos = v.aux(layer, 0);
    uint32_t slot = 0, slph = 0;
    bool ok = true;
    int4 e = w0 < total ? klist[KSTEP * w0] : kt_none;
    int pos_cur = w0 < total ? kpos[(size_t)e.x * TILE + row] : 0;
    // the row of the score scratch this token's scores go to: its V slot (rows past the tile's last token have none)
    int vrow_cur = w0 < total && row < (e.y >> 8) ? v.kv_link[(size_t)e.x * TILE + row] : 0;
    for (int w = w0; w < total && ok; ++w) {
      const int4 nxt = w + 1 < total ? klist[KSTEP * (w + 1)] : kt_none;
      const int cls = e.y & 0x7f, n_valid = e.y >> 8, qs = e.w;
      const bool discard = (e.y & KE_DISCARD) != 0;
      const int passes = (cls + KT_A_SLOTS - 1) / KT_A_SLOTS;
      const int pos_next = nxt.w >= 0 ? kpos[(size_t)nxt.x * TILE + row] : 0;
      const int vrow_next = nxt.w >= 0 && row < (nxt.y >> 8) ? v.kv_link[(size_t)nxt.x * TILE + row] : 0;
      const bool has_row = row < n_valid;
      float* const out_row = v.scores + (size_t)vrow_cur * Hq;
      // a row counts if it holds a token and, for a causal (prefill) query, the token is not after the query
      const int pos_limit = v.qpos ? v.qpos[qs] : 0x7fffffff;
      const bool live = row < n_valid && pos_cur <= pos_limit;
      for (int ps = 0; ps < passes && ok; ++ps) {
        const uint32_t mode = discard ? KP_DISCARD : passes == 1 ? KP_STORE_FINAL : (ps == 0 ? KP_STORE_PART : KP_ADD_FINAL);
        for (int sli = 0; sli < Hkv; ++sli) {
          const int g = sli + g_rot < Hkv ? sli + g_rot : sli + g_rot - Hkv;
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(s_full + 8 * slot, slph, abort_flag)))) break;
          fence_after_sync();
          float sv[REP];
          {
            uint32_t* dst = reinterpret_cast<uint32_t*>(sv);
            const uint32_t src = lane_addr + s_col0 + 16 * slot;
            if constexpr (REP == 1) tmem_ld1(src, dst);
            else if constexpr (REP == 2) tmem_ld2(src, dst);
            else if constexpr (REP == 4) tmem_ld4(src, dst);
            else tmem_ld8(src, dst);
          }
          tmem_ld_wait();
          fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(s_empty_own + 8 * slot);
            else mbar_arrive(s_empty + 8 * slot);
          }
          if (++slot == (uint32_t)KT_S_SLOTS) { slot = 0; slph ^= 1u; }
          if (mode == KP_DISCARD) continue;
          float* out = out_row + g * REP;
#pragma unroll
          for (int i = 0; i < REP; ++i) {
            float x = sv[i] * sm_scale;
            if (mode == KP_ADD_FINAL && has_row) x += out[i];                            // the first pass stored its part
            sv[i] = live ? x : -INFINITY;
          }
          if (has_row) {
            if constexpr (REP >= 4) {
#pragma unroll
              for (int i = 0; i < REP; i += 4) *reinterpret_cast<float4*>(out + i) = make_float4(sv[i], sv[i + 1], sv[i + 2], sv[i + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < REP; ++i) out[i] = sv[i];
            }
          }
          if (mode != KP_STORE_PART) {
            unsigned mine = 0u;
#pragma unroll
            for (int i = 0; i < REP; ++i) {
              const unsigned m = warp_max_u32(enc_ordered(sv[i]));
              if (lane == i) mine = m;
            }
            if (lane < REP) atomicMax(&v.seqmax[qs * Hq + g * REP + lane], mine);
          }
        }
      }
      pos_cur = pos_next;
      vrow_cur = vrow_next;
      e = nxt;
    }
    tmem_ld_wait();                                                          // nothing of this thread is in flight when TMEM is freed
  }

  fence_before_sync();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();                       // the partner is done with this CTA's memory and barriers as well
  fence_after_sync();
  if (warp == 1) {
    if constexpr (PAIR) tmem_dealloc_pair(tmem_base, KT_TMEM_COLS);
    else tmem_dealloc(tmem_base, KT_TMEM_COLS);
  }
  if (tid == 0 && *abort_flag) set_status(v, misaligned ? TWKV_ERR_DEVICE_CHECK : TWKV_ERR_TIMEOUT);
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
// One TMA box then reads 16 KiB of consecutive lines (a half panel for the CTA-pair kernel: rows 0..63 or 64..127).
__global__ void uinv_panels_kernel(const unsigned short* __restrict__ in, unsigned short* __restrict__ out, int d) {
  __shared__ unsigned short t[64][129];
  const int j64 = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
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
  uinv_panels_kernel<<<dim3(d / 64, d / 128), 256, 0, st>>>(reinterpret_cast<const unsigned short*>(in),
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

size_t kscore_tc_smem_bytes(int nb, size_t stage_bytes) {
  return (size_t)KT_A_SLOTS * PANEL_BYTES + (size_t)nb * stage_bytes + 2 * KT_Q_PANEL_BYTES + KT_ROPE_STAGE_BYTES + 8 * (KT_N_BARS + 2 * nb) +
         2 * sizeof(int);
}
constexpr int KT_NB_SINGLE = 2, KT_NB_PAIR = 4;                // ring stages of two U_K^-1 panels (32 KiB) / two half panels (16 KiB)

// CTA pairs of the pair kernel that can be resident at once on the current device (0: it cannot run).
static int kscore_query_pairs(int sm_count) {
  const size_t smem = kscore_tc_smem_bytes(KT_NB_PAIR, PANEL_BYTES);
  if (cudaFuncSetAttribute(kscore_tc_kernel<false, 4, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) { cudaGetLastError(); return 0; }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(KT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.gridDim = dim3(sm_count & ~1);
  cudaLaunchAttribute pair_attr;
  pair_attr.id = cudaLaunchAttributeClusterDimension;
  pair_attr.val.clusterDim.x = 2; pair_attr.val.clusterDim.y = 1; pair_attr.val.clusterDim.z = 1;
  cfg.attrs = &pair_attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kscore_tc_kernel<false, 4, true, false>, &cfg) != cudaSuccess || n < 1) { cudaGetLastError(); n = 0; }
  return n;
}
int kscore_max_pairs(int sm_count) {
  static const int cached = kscore_query_pairs(sm_count);       // queried once per process (thread-safe initialisation)
  return cached;
}

template <bool BF16, bool PAIR, bool DBG>
static cudaError_t launch_kscore_tc_t(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                                      const void* q, int n_pieces, cudaStream_t st) {
  const int nb = PAIR ? KT_NB_PAIR : KT_NB_SINGLE;
  const size_t smem = kscore_tc_smem_bytes(nb, PAIR ? PANEL_BYTES : 2 * PANEL_BYTES);
  const unsigned short* qq = reinterpret_cast<const unsigned short*>(q);
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(KT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.gridDim = dim3(PAIR ? 2 * n_pieces : n_pieces);
  cudaLaunchAttribute pair_attr;
  pair_attr.id = cudaLaunchAttributeClusterDimension;
  pair_attr.val.clusterDim.x = 2; pair_attr.val.clusterDim.y = 1; pair_attr.val.clusterDim.z = 1;
  cfg.attrs = PAIR ? &pair_attr : nullptr;
  cfg.numAttrs = PAIR ? 1 : 0;
  ProfScope ps(TWKV_K_KSCORE, st);
  cudaError_t e = cudaSuccess;
#define TWKV_KT(REP)                                                                                                  \
  {                                                                                                                   \
    e = cudaFuncSetAttribute(kscore_tc_kernel<BF16, REP, PAIR, DBG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                                   \
    e = cudaLaunchKernelEx(&cfg, kscore_tc_kernel<BF16, REP, PAIR, DBG>, map_blocks, map_uinvT, v, layer, qq, nb);        \
  }
  switch (v.rep) {
    case 1: TWKV_KT(1) break;
    case 2: TWKV_KT(2) break;
    case 4: TWKV_KT(4) break;
    default: TWKV_KT(8) break;
  }
#undef TWKV_KT
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

// `pairs`: run on CTA pairs (n_pieces pairs, map_uinvT with 64-row boxes) instead of single CTAs (128-row boxes).
cudaError_t launch_kscore_tc(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                             const void* q, int n_pieces, bool pairs, cudaStream_t st) {
#define TWKV_KS_LAUNCH(BF, PR)                                                                                  \
  (v.debug ? launch_kscore_tc_t<BF, PR, true>(v, layer, map_blocks, map_uinvT, q, n_pieces, st)                 \
           : launch_kscore_tc_t<BF, PR, false>(v, layer, map_blocks, map_uinvT, q, n_pieces, st))
  if (pairs) return v.dtype == TWKV_BF16 ? TWKV_KS_LAUNCH(true, true) : TWKV_KS_LAUNCH(false, true);
  return v.dtype == TWKV_BF16 ? TWKV_KS_LAUNCH(true, false) : TWKV_KS_LAUNCH(false, false);
#undef TWKV_KS_LAUNCH
}

}  // namespace twkv
