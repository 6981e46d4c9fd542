// V-side of decode attention on the 5th-generation tensor cores.
//
// By linearity of Eq. 3 the weighted sum of the values is taken in spectral space: per (query slot, split, head group)
//   acc[j][h] = sum over the split's tokens t of  X^_V[t][j] * p[t][h],   p = exp(s - max) rounded to the cache dtype,
//   l[h]      = sum over t of p[t][h],
// and merge_kernel projects acc / l through U_V^-1 once.  A V tile of rank class c is c panels [128 tokens x 64
// columns] in HBM.  Two panels at a time form the A operand of one tcgen05.mma chain (M = 128 spectral columns, N = the
// CTA's heads padded to 16 / 32, K = 16 tokens per instruction, 8 instructions per tile): a panel as TMA lands it
// (rows of 128 bytes, 128-byte swizzle) is exactly the MN-major operand layout, the second panel of the pair being the
// second 64-column atom along M (leading byte offset = one panel).  The fp32 accumulator of panel pair i is N columns of
// TMEM at column i * N and stays there for the whole kernel; no accumulator lives in registers and the panels are read
// from shared memory by the tensor core only.  A class with an odd number of panels ends with a lone panel; its chain
// points the second atom at a small zero block instead (the leading byte offset is free per instruction), so the pair's
// upper accumulator half adds zeros.
// The probabilities are the B operand (K-major: [head][token], two 64-token halves), written by 8 warps: thread =
// (head, 8 consecutive tokens), one 16-byte swizzled store per 8 weights.  The K-score kernel stores a token's scores at
// its V slot, so a tile's 128 score rows lie next to each other: one TMA box [128 rows x the CTA's heads] per tile,
// issued by the producer thread two tiles ahead into a ring of four tiles in shared memory (TS = true).  A narrow tile
// reads as many bytes of scores as of values, and with one tile in flight their latency bound the kernel.  Where the
// head count is not a multiple of four (rows not 16-byte aligned: no tensor map) each warp copies the rows of its own
// token groups with cp.async instead (TS = false).
// bf16 weights go in as two bf16 parts (see below), two chains per pair.
//
// Warp roles (320 threads, one CTA per SM):
//   warp 0      TMA producer of V panels (ring of 32-KiB pair stages; one elected lane)
//   warp 1      MMA issuer (one elected lane; owns the TMEM allocation)
//   warps 2-9   probabilities, then at the end the read-out of the accumulators to the split's partial result
// All waits are bounded (tc_util.cuh); a wait that runs out ends the kernel with TWKV_ERR_TIMEOUT.
#include "twkv_dev.h"
#include "tc_util.cuh"
#include "mma_util.cuh"

namespace twkv {
using namespace tc;

constexpr int VT_PWARPS = 8;
constexpr int VT_PTHREADS = 32 * VT_PWARPS;
constexpr int VT_THREADS = 64 + VT_PTHREADS;
constexpr int VT_META = 256;                                   // tiles whose descriptors are staged in shared memory at a time
constexpr uint32_t VT_PANEL_BYTES = 16384;
constexpr uint32_t VT_STAGE_BYTES = 2 * VT_PANEL_BYTES;
constexpr uint32_t VT_ZERO_BYTES = 2048;                       // 16 token rows of zeros: the missing partner of a lone panel
constexpr uint32_t VT_SMEM_MAX = 232448;
constexpr int VT_SC = 4;                                       // tiles of scores in flight

template <bool BF16, int N>
struct VtCfg {
  static constexpr int PARTS = BF16 ? 2 : 1;                   // operands per weight
  static constexpr uint32_t P_HALF_BYTES = N * 128;            // [N heads][64 tokens]
  static constexpr uint32_t P_PART_BYTES = 2 * P_HALF_BYTES;
  static constexpr uint32_t P_BUF_BYTES = PARTS * P_PART_BYTES;
  static constexpr uint32_t TAIL_BYTES = VT_META * 16 + VT_PTHREADS * 4 + 256;      // descriptors, row sums, barriers
  static constexpr uint32_t SC_STAGE_BYTES = 128 * N * 4;      // [128 tokens][N heads] fp32
  static constexpr uint32_t FIXED_BYTES = VT_ZERO_BYTES + 2 * P_BUF_BYTES + VT_SC * SC_STAGE_BYTES + TAIL_BYTES + 1024;   // + alignment slack
  static constexpr int STAGES_FIT = (int)((VT_SMEM_MAX - FIXED_BYTES) / VT_STAGE_BYTES);
  static constexpr int STAGES = STAGES_FIT < 6 ? STAGES_FIT : 6;
  static constexpr uint32_t SMEM_BYTES = STAGES * VT_STAGE_BYTES + FIXED_BYTES;
  static constexpr int ITEMS = N / 16;                         // (head, 8-token group) items per probability thread and tile
};

// Two fp32 -> one packed pair in the cache dtype (a in the low half), round to nearest; r0 / r1: the rounded values.
template <bool BF16> __device__ __forceinline__ uint32_t vt_pack2(float a, float b, float& r0, float& r1) {
  uint32_t d;
  if constexpr (BF16) {
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
    r0 = __uint_as_float(d << 16);
    r1 = __uint_as_float(d & 0xffff0000u);
  } else {
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&d));
    r0 = f.x; r1 = f.y;
  }
  return d;
}

// Instruction descriptor: kind::f16, fp32 accumulate, A MN-major (bit 15), B K-major, M = 128.
__host__ __device__ constexpr uint32_t vt_idesc(int fmt, int n) { return idesc_f16(fmt, 128, n) | (1u << 15); }

template <bool BF16, int N, bool TS>
__global__ void __launch_bounds__(VT_THREADS, 1)
vacc_tc_kernel(const __grid_constant__ CUtensorMap map_blocks, const __grid_constant__ CUtensorMap map_scores, DevView v, int layer,
               const int* __restrict__ seq_ids, int n_splits) {
  using C = VtCfg<BF16, N>;
  constexpr int S = C::STAGES, PARTS = C::PARTS, ITEMS = C::ITEMS;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hq = v.Hq, d_kv = v.d_kv;
  const int qs = blockIdx.x / n_splits, split = blockIdx.x - qs * n_splits;
  const int h0 = blockIdx.y * N, nh = min(N, Hq - h0);
  const int NB = min(N, Hq);                                    // heads per score row in shared memory (TS: the box's width)
  const int seq = seq_ids[qs];
  const bool seq_ok = seq >= 0 && seq < v.S;
  // this split's range of the sequence's V tile list in stride order, cut by plan_kernel to equal cost; an id outside
  // the cache has no tiles and contributes nothing: zero partials
  const int* cut = v.vcut + (size_t)qs * (n_splits + 1) + split;
  const int t_first = cut[0], n_mine = seq_ok ? cut[1] - t_first : 0;
  const int n_tiles = seq_ok ? v.svc(layer)[seq] : 0;
  const long long t_stride = vtile_stride(n_tiles);
  const int* list = v.svt(layer) + (size_t)(seq_ok ? seq : 0) * v.TPS;
  const int4* desc = v.desc(layer, 1);

  // shared memory: ring | zero block | probabilities [2 buffers][PARTS][2 halves][N][128 B] | score ring | descriptors | row sums | barriers
  const uint32_t s0 = smem_addr(smem_raw);
  const uint32_t pad = (1024u - (s0 & 1023u)) & 1023u;          // operand tiles need 1024-byte alignment for the swizzle
  unsigned char* base_ptr = smem_raw + pad;
  const uint32_t sRing = s0 + pad;
  const uint32_t sZero = sRing + S * VT_STAGE_BYTES;
  const uint32_t sP = sZero + VT_ZERO_BYTES;
  unsigned char* sP_ptr = base_ptr + S * VT_STAGE_BYTES + VT_ZERO_BYTES;
  unsigned char* sS_ptr = sP_ptr + 2 * C::P_BUF_BYTES;                                // score ring
  const uint32_t sS = sP + 2 * C::P_BUF_BYTES;
  int4* s_meta = reinterpret_cast<int4*>(sS_ptr + VT_SC * C::SC_STAGE_BYTES);          // (tile, class, tokens, first block)
  float* s_l = reinterpret_cast<float*>(s_meta + VT_META);
  unsigned char* tail = reinterpret_cast<unsigned char*>(s_l + VT_PTHREADS);
  const uint32_t bars = smem_addr(tail);
  const uint32_t full = bars, empty = full + 8 * S, p_full = empty + 8 * S, p_empty = p_full + 16, acc_done = p_empty + 16;
  const uint32_t sc_full = acc_done + 8, sc_empty = sc_full + 8 * VT_SC;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(tail + 8 * (2 * S + 5 + 2 * VT_SC));
  volatile int* abort_flag = reinterpret_cast<int*>(s_tmem_base + 1);

  const int n_pairs = (v.NC + 1) >> 1;
  uint32_t tmem_cols = 32;
  while (tmem_cols < (uint32_t)(n_pairs * N)) tmem_cols <<= 1;

  if (tid == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(full + 8 * i, 1); mbar_init(empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(p_full + 8 * i, VT_PWARPS); mbar_init(p_empty + 8 * i, 1); }
    mbar_init(acc_done, 1);
    for (int i = 0; i < VT_SC; ++i) { mbar_init(sc_full + 8 * i, 1); mbar_init(sc_empty + 8 * i, VT_PWARPS); }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(smem_addr(s_tmem_base), tmem_cols);
  for (int i = tid; i < (int)VT_ZERO_BYTES / 16; i += VT_THREADS)
    reinterpret_cast<uint4*>(base_ptr + S * VT_STAGE_BYTES)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *s_tmem_base;

  // role state that survives the descriptor chunks
  uint32_t st = 0, st_ph = 0;                                   // producer / issuer: ring stage and its phase
  uint32_t n_loaded = 0;                                        // producer: stages filled so far
  uint32_t n_boxes = 0;                                         // producer: score boxes requested so far
  uint32_t touched = 0;                                         // issuer: panel pairs whose accumulator holds a value
  bool ok = true;
  int max_cls = 0;                                              // probability warps: widest class seen (which accumulators to read)
  float l_sum = 0.f;                                            // probability threads: sum of this thread's weights

  // probability threads: fixed head, items = 8-token groups
  const int pt = tid - 64;                                      // 0 .. 255 for warps 2-9
  const int ph_ = pt & (N - 1);                                 // head within the CTA's group
  float m_h = 0.f;
  if (warp >= 2) {
    // a query that sees no token (chunked prefill, every cached position after its own) has no maximum: weights stay 0
    const float m = ph_ < nh ? dec_ordered(v.seqmax[qs * Hq + h0 + ph_]) : 0.f;
    m_h = m == -INFINITY ? 0.f : m;
  }

  for (int c0 = 0; c0 < n_mine; c0 += VT_META) {
    const int cn = min(VT_META, n_mine - c0);
    // descriptors of this chunk of the split's tiles
    for (int i = tid; i < cn; i += VT_THREADS) {
      const int t = list[(int)(((long long)(t_first + c0 + i) * t_stride) % n_tiles)];
      const int4 d = desc[t];
      s_meta[i] = make_int4(t, d.y, d.z, d.w);
    }
    __syncthreads();

    if (warp == 0) {
      // ------------------------------------------------------------- TMA producer
      if (elect_one()) {
        if (c0 == 0) { tma_prefetch_desc(&map_blocks); if constexpr (TS) tma_prefetch_desc(&map_scores); }
        // the score rows of tile i of the chunk: one box [128 rows x NB heads] into stage (c0 + i) % VT_SC
        auto score_box = [&](int i) -> bool {
          const uint32_t k = (uint32_t)(c0 + i), stg = k % VT_SC;
          if (!mbar_wait_thin(sc_empty + 8 * stg, ((k / VT_SC) & 1u) ^ 1u, abort_flag)) return false;
          mbar_expect_tx(sc_full + 8 * stg, (uint32_t)(TILE * NB * 4));
          tma_load_2d(sS + stg * C::SC_STAGE_BYTES, &map_scores, sc_full + 8 * stg, h0, s_meta[i].x * TILE);
          n_boxes = k + 1;
          return true;
        };
        if constexpr (TS) {
          for (int i = 0; i < 2 && i < cn && ok; ++i) ok = score_box(i);
        }
        for (int i = 0; i < cn && ok; ++i) {
          const int4 m = s_meta[i];
          if constexpr (TS) {
            if (i + 2 < cn && !(ok = score_box(i + 2))) break;
          }
          for (int j = 0; j < m.y; j += 2) {
            if (!(ok = mbar_wait_thin(empty + 8 * st, st_ph ^ 1u, abort_flag))) break;
            const bool two = j + 1 < m.y;
            mbar_expect_tx(full + 8 * st, two ? VT_STAGE_BYTES : VT_PANEL_BYTES);
            tma_load_2d(sRing + st * VT_STAGE_BYTES, &map_blocks, full + 8 * st, 0, (m.w + j) * TILE);
            if (two) tma_load_2d(sRing + st * VT_STAGE_BYTES + VT_PANEL_BYTES, &map_blocks, full + 8 * st, 0, (m.w + j + 1) * TILE);
            ++n_loaded;
            if (++st == (uint32_t)S) { st = 0; st_ph ^= 1u; }
          }
        }
        if (!ok) {                                              // let copies in flight land before the CTA goes away
          for (uint32_t i = 0; i < (uint32_t)S && i < n_loaded; ++i) {
            const uint32_t n = n_loaded - 1 - i;
            mbar_wait_drain(full + 8 * (n % S), (n / S) & 1u);
          }
          for (uint32_t i = 0; i < (uint32_t)VT_SC && i < n_boxes; ++i) {
            const uint32_t n = n_boxes - 1 - i;
            mbar_wait_drain(sc_full + 8 * (n % VT_SC), (n / VT_SC) & 1u);
          }
        }
      }
      __syncwarp();
    } else if (warp == 1) {
      // ------------------------------------------------------------- MMA issuer
      if (elect_one()) {
        constexpr uint32_t idesc = vt_idesc(BF16 ? 1 : 0, N);
        for (int i = 0; i < cn && ok; ++i) {
          const int k = c0 + i;
          const int cls = s_meta[i].y;
          const uint32_t buf = (uint32_t)k & 1u;
          if (!(ok = mbar_wait_thin(p_full + 8 * buf, ((uint32_t)k >> 1) & 1u, abort_flag))) break;
          const uint32_t pb = sP + buf * C::P_BUF_BYTES;
          for (int j = 0; j < cls; j += 2) {
            if (!(ok = mbar_wait_thin(full + 8 * st, st_ph, abort_flag))) break;
            fence_after_sync();
            const uint32_t a0 = sRing + st * VT_STAGE_BYTES;
            const bool two = j + 1 < cls;
            const uint32_t pair = (uint32_t)j >> 1, d_tmem = tmem_base + pair * N;
            uint32_t acc = (touched >> pair) & 1u;
#pragma unroll
            for (int part = 0; part < PARTS; ++part) {
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const uint32_t a_addr = a0 + ks * 2048u;                                   // 16 token rows per instruction
                const uint32_t lbo = two ? VT_PANEL_BYTES : sZero - a_addr;               // where the second 64 columns are
                const uint32_t a_lo = ((a_addr >> 4) & 0x3fffu) | ((lbo >> 4) << 16);
                const uint32_t b_addr = pb + part * C::P_PART_BYTES + (ks >> 2) * C::P_HALF_BYTES + (ks & 3) * 32u;
                const uint32_t b_lo = kmajor_sw128_desc_lo(b_addr);
                const uint64_t ad = ((uint64_t)KMAJOR_SW128_DESC_HI << 32) | a_lo, bd = ((uint64_t)KMAJOR_SW128_DESC_HI << 32) | b_lo;
                mma_f16_ss(d_tmem, ad, bd, idesc, acc);
                acc = 1u;
              }
            }
            touched |= 1u << pair;
            mma_commit(empty + 8 * st);
            if (++st == (uint32_t)S) { st = 0; st_ph ^= 1u; }
          }
          if (!ok) break;
          mma_commit(p_empty + 8 * buf);
        }
        if (ok && c0 + cn == n_mine) mma_commit(acc_done);
      }
      __syncwarp();
    } else {
      // ------------------------------------------------------------- probabilities
      // One cp.async group per iteration: the score rows of tile i + VT_SC - 1.  Waiting for all but the newest
      // VT_SC - 1 groups then guarantees tile i's scores.  A warp copies and reads only the rows of its own token groups.
      constexpr int GL = N == 16 ? 16 : 32;                     // lanes that share an item
      const int gl = lane & (GL - 1);
      const bool al16 = (Hq & 3) == 0;                          // score rows start on 16-byte boundaries
      // Starts the copies of tile i's score rows into its stage of the score ring.  Every row of the stage is written:
      // rows past the tile's last token, and heads past the CTA's last, get -inf (weight 0).
      auto issue_scores = [&](int i) {
        if (i < cn) {
          const uint32_t stage = (uint32_t)((c0 + i) % VT_SC) * C::SC_STAGE_BYTES;
          const int4 m = s_meta[i];
          const int n_valid = m.z;
          const float* rows = v.scores + (size_t)m.x * TILE * Hq + h0;            // the tile's first score row, at this CTA's heads
          if (al16) {
            constexpr int CPR = N / 4, R = 8 * CPR / GL;        // 16-byte pieces per row; pieces per lane and item
#pragma unroll
            for (int it = 0; it < ITEMS; ++it)
#pragma unroll
              for (int r = 0; r < R; ++r) {
                const int row = ((it * VT_PTHREADS + pt) / N) * 8 + (r * GL + gl) / CPR, ch = (r * GL + gl) % CPR;
                const uint32_t off = stage + (uint32_t)((row * N + 4 * ch) * 4);
                if (row < n_valid && 4 * ch < nh) cp_async16(sS + off, rows + (size_t)row * Hq + 4 * ch);
                else *reinterpret_cast<float4*>(sS_ptr + off) = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
              }
          } else {
            constexpr int R = 8 * N / GL;
#pragma unroll
            for (int it = 0; it < ITEMS; ++it)
#pragma unroll
              for (int r = 0; r < R; ++r) {
                const int row = ((it * VT_PTHREADS + pt) / N) * 8 + (r * GL + gl) / N, hh = (r * GL + gl) % N;
                const uint32_t off = stage + (uint32_t)((row * N + hh) * 4);
                if (row < n_valid && hh < nh) cp_async4(sS + off, rows + (size_t)row * Hq + hh);
                else *reinterpret_cast<float*>(sS_ptr + off) = -INFINITY;
              }
          }
        }
      };
      if constexpr (!TS) {
#pragma unroll 1
        for (int d = 0; d < VT_SC - 1; ++d) { issue_scores(d); cp_async_commit(); }
      }
      for (int i = 0; i < cn && ok; ++i) {
        const int k = c0 + i;
        max_cls = max(max_cls, s_meta[i].y);
        const int n_valid_i = s_meta[i].z;
        if constexpr (TS) {
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(sc_full + 8 * ((uint32_t)k % VT_SC), ((uint32_t)k / VT_SC) & 1u, abort_flag)))) break;
        } else {
          issue_scores(i + VT_SC - 1);
          cp_async_commit();
          cp_async_wait<VT_SC - 1>();                           // this thread's copies of tile i have landed
          __syncwarp();                                         // ... and the other lanes'
        }
        const uint32_t buf = (uint32_t)k & 1u;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(p_empty + 8 * buf, (((uint32_t)k >> 1) & 1u) ^ 1u, abort_flag)))) break;
        unsigned char* pb = sP_ptr + buf * C::P_BUF_BYTES;
        const float* srow = reinterpret_cast<const float*>(sS_ptr + (uint32_t)(k % VT_SC) * C::SC_STAGE_BYTES) + ph_;
        const int rs = TS ? NB : N;                             // floats per score row in the stage
        // a box holds whatever the scratch holds in rows past the tile's last token and has no columns past the last head
        const bool head_ok = !TS || ph_ < nh;
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
          const int tg = (it * VT_PTHREADS + pt) / N;
          uint32_t hi[4];
          [[maybe_unused]] uint32_t lo[4];
#pragma unroll
          for (int u = 0; u < 8; u += 2) {
            float p0 = __expf(srow[(tg * 8 + u) * rs] - m_h), p1 = __expf(srow[(tg * 8 + u + 1) * rs] - m_h);
            if constexpr (TS) {
              p0 = (head_ok && tg * 8 + u < n_valid_i) ? p0 : 0.f;
              p1 = (head_ok && tg * 8 + u + 1 < n_valid_i) ? p1 : 0.f;
            }
            // two weights per conversion instruction (single conversions run at a quarter of the rate and bound this loop)
            float r0, r1;
            hi[u >> 1] = vt_pack2<BF16>(p0, p1, r0, r1);
            l_sum += r0 + r1;
            if constexpr (BF16) {
              // bf16 keeps 8 bits of a weight: with few tokens per sequence that rounding alone reaches 1e-3 of the
              // output, so the remainder goes into a second operand (16 bits in all)
              float q0, q1;
              lo[u >> 1] = vt_pack2<true>(p0 - r0, p1 - r1, q0, q1);
              l_sum += q0 + q1;
            }
          }
          const uint32_t off = (uint32_t)(tg >> 3) * C::P_HALF_BYTES + (uint32_t)ph_ * 128u + ((((uint32_t)tg & 7u) ^ ((uint32_t)ph_ & 7u)) << 4);
          *reinterpret_cast<uint4*>(pb + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          if constexpr (BF16) *reinterpret_cast<uint4*>(pb + C::P_PART_BYTES + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
        fence_proxy_async_smem();
        __syncwarp();                                           // also: the stage is read before the next copies into it start
        if (lane == 0) {
          mbar_arrive(p_full + 8 * buf);
          if constexpr (TS) mbar_arrive(sc_empty + 8 * ((uint32_t)k % VT_SC));
        }
      }
      if constexpr (!TS) cp_async_wait<0>();
    }
    __syncthreads();                                            // the descriptors may be replaced
    ok = ok && !*abort_flag;
  }

  // ----------------------------------------------------------------- partial results of this split
  const size_t pidx = (size_t)qs * n_splits + split;
  if (warp >= 2) {
    s_l[pt] = l_sum;
    bool ready = ok;
    if (ready && n_mine > 0) ready = __all_sync(0xffffffffu, mbar_wait(acc_done, 0u, abort_flag));
    fence_after_sync();
    float* pa = v.part_acc + pidx * Hq * d_kv;
    const int quad = warp & 3;                                  // the TMEM lanes this warp may read
    const int used_pairs = ready ? (max_cls + 1) >> 1 : 0;
    for (int pair = (warp - 2) >> 2; pair < n_pairs; pair += 2) {
      const int col = pair * 128 + quad * 32 + lane;            // spectral column of this thread's TMEM lane
      const bool used = pair < used_pairs;
      const uint32_t src = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(pair * N);
#pragma unroll 1
      for (int n0 = 0; n0 < N; n0 += 16) {                      // sixteen heads at a time
        float val[16];
        if (used) {
          tmem_ld16(src + n0, reinterpret_cast<uint32_t*>(val));
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int n = 0; n < 16; ++n) val[n] = 0.f;
        }
        if (col < d_kv) {
          float* dst = pa + (size_t)(h0 + n0) * d_kv + col;
#pragma unroll
          for (int n = 0; n < 16; ++n)
            if (n0 + n < nh) dst[(size_t)n * d_kv] = val[n];
        }
      }
    }
    tmem_ld_wait();
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
  if (tid < nh) {
    // row sums: this head's probability threads in index order
    float l = 0.f;
    for (int i = tid; i < VT_PTHREADS; i += N) l += s_l[i];
    v.part_l[pidx * Hq + h0 + tid] = l;
  }
  if (tid == 0 && *abort_flag) set_status(v, TWKV_ERR_TIMEOUT);
}

template <bool BF16, int N, bool TS>
static cudaError_t launch_vacc_tc_n(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_scores,
                                    const int* seq_ids, int n_seq, int n_splits, cudaStream_t st) {
  using C = VtCfg<BF16, N>;
  static_assert(C::STAGES >= 3, "the ring needs a few stages");
  cudaError_t e = cudaFuncSetAttribute(vacc_tc_kernel<BF16, N, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const dim3 grid(n_seq * n_splits, (v.Hq + N - 1) / N);
  vacc_tc_kernel<BF16, N, TS><<<grid, VT_THREADS, C::SMEM_BYTES, st>>>(map_blocks, map_scores, v, layer, seq_ids, n_splits);
  return cudaGetLastError();
}

// map_scores: the score scratch as a tensor map (boxes of 128 rows x min(N, Hq) heads), or null: rows copied with cp.async.
cudaError_t launch_vacc_tc(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap* map_scores, const int* seq_ids,
                           int n_seq, int n_splits, cudaStream_t st) {
  const bool bf16 = v.dtype == TWKV_BF16;
  // up to 32 heads per CTA; more heads run as further CTAs that read the same panels (through L2)
#define TWKV_VT(BF, NN)                                                                                                   \
  (map_scores ? launch_vacc_tc_n<BF, NN, true>(v, layer, map_blocks, *map_scores, seq_ids, n_seq, n_splits, st)           \
              : launch_vacc_tc_n<BF, NN, false>(v, layer, map_blocks, map_blocks, seq_ids, n_seq, n_splits, st))
  if (v.Hq <= 16) return bf16 ? TWKV_VT(true, 16) : TWKV_VT(false, 16);
  return bf16 ? TWKV_VT(true, 32) : TWKV_VT(false, 32);
#undef TWKV_VT
}

}  // namespace twkv
