// Decode attention over the mixed-rank cache (Eq. 3, reshape to heads, RoPE, softmax attention).
//
//   plan_kernel    sequence id -> query slot map, running-max reset, K-tile work list
//   kscore_tc_kernel (kscore_tc.cu)  per K tile: Kbar = X^_K U_K^-1, RoPE by stored position,
//                  s = q . Kbar * scale for the GQA group, scores to scratch, per-sequence max
//   vacc_kernel    per (sequence, split): p = exp(s - max), acc += p^T X^_V in spectral space
//                  (tensor cores), l = sum p
//   merge_kernel   sum of the splits, out_h = (acc_h / l_h) U_V^-1[:, head slice]
//
// V is never reconstructed per token: by linearity of Eq. 3 the weighted sum is taken in
// spectral space and projected once.
#include <type_traits>
#include "twkv_dev.h"
#include "mma_util.cuh"
#include "tc_util.cuh"

namespace twkv {

// ------------------------------------------------------------------------------ plan
// One CTA: sequence id -> query slot map, running-max reset, and the K-score work list: the K tiles
// of the listed sequences in class order (widest first, inside a class in table order), compacted
// with block-wide scans so the order does not depend on thread timing.  For the CTA-pair kernel the list
// is rewritten as items of two tiles of one class.  The list is then cut into n_cta contiguous pieces of
// about equal estimated cost, so a CTA (pair) of the K-score kernel mostly stays inside one (class, sequence) run.
__device__ __forceinline__ unsigned ktile_cost(int cls) {
  // cycles per tile of the K-score kernel by rank class, measured inside the kernel on the benchmark's mix of classes
  // (8 KV heads, CTA pairs): a fixed part (rotation factors, the per-slab epilogue and score products) plus a per-panel
  // part; classes above 8 run as two passes.  Only the ratios matter.
  constexpr unsigned kCost[TWKV_MAX_CLASSES] = {16300u, 17800u, 18900u, 19500u, 20900u, 21900u, 23900u, 24300u,
                                                39800u, 39800u, 40700u, 41100u, 42400u, 42900u, 45000u, 46700u};
  return kCost[min(max(cls, 1), TWKV_MAX_CLASSES) - 1];
}

__global__ void __launch_bounds__(1024) plan_kernel(DevView v, int layer, const int* __restrict__ seq_ids, int n_seq, int n_cta, int pairs) {
  __shared__ int s_cls_off[TWKV_MAX_CLASSES + 1];
  __shared__ unsigned s_wsum[32];
  __shared__ unsigned s_base;                                     // entries kept so far
  __shared__ int s_keep[TWKV_MAX_CLASSES];                        // kept tiles per class run (run k = class NC - k)
  __shared__ int s_koff[TWKV_MAX_CLASSES + 1], s_ioff[TWKV_MAX_CLASSES + 1];    // start of run k in the tile list / in the item list
  __shared__ unsigned long long s_coff[TWKV_MAX_CLASSES + 1];     // estimated cost of everything before run k
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int s = tid; s < v.S; s += blockDim.x) v.qslot[s] = -1;
  if (tid < TWKV_MAX_CLASSES) s_keep[tid] = 0;
  if (tid == 0) {
    const int* kcc = v.kcc(layer);
    int run = 0;
    for (int c = v.NC; c >= 1; --c) { s_cls_off[v.NC - c] = run; run += kcc[c - 1]; }    // widest class first
    s_cls_off[v.NC] = run;
    s_base = 0u;
  }
  __syncthreads();
  for (int i = tid; i < n_seq; i += blockDim.x) {
    const int s = seq_ids[i];
    if (s < 0 || s >= v.S) set_status(v, TWKV_ERR_INVALID_ARG);
    else v.qslot[s] = i;
  }
  for (int i = tid; i < n_seq * v.Hq; i += blockDim.x) v.seqmax[i] = 0u;
  __syncthreads();
  for (int i = tid; i < n_seq; i += blockDim.x) {
    const int s = seq_ids[i];
    if (s >= 0 && s < v.S && v.qslot[s] != i) set_status(v, TWKV_ERR_INVALID_ARG);   // duplicate id
  }
  const int4* desc = v.desc(layer, 0);
  const int* kct = v.kct(layer);
  const int n_all = s_cls_off[v.NC];
  constexpr int PL_BATCH = 4;                                     // list chunks of 1024 whose table reads are issued together
  for (int f0 = 0; f0 < n_all; f0 += 1024 * PL_BATCH) {
    // the three dependent reads (tile id -> descriptor -> query slot) of PL_BATCH chunks go out level by level
    int tile[PL_BATCH], run_[PL_BATCH];
    int4 d[PL_BATCH];
    int4 ent[PL_BATCH];
#pragma unroll
    for (int u = 0; u < PL_BATCH; ++u) {
      const int f = f0 + u * 1024 + tid;
      tile[u] = -1; run_[u] = 0;
      if (f < n_all) {
        int k = 0;
        while (f >= s_cls_off[k + 1]) ++k;
        run_[u] = k;
        tile[u] = kct[(size_t)(v.NC - k - 1) * v.NT + (f - s_cls_off[k])];
      }
    }
#pragma unroll
    for (int u = 0; u < PL_BATCH; ++u) d[u] = tile[u] >= 0 ? desc[tile[u]] : make_int4(0, 0, 0, 0);
#pragma unroll
    for (int u = 0; u < PL_BATCH; ++u)
      ent[u] = tile[u] >= 0 ? make_int4(tile[u], d[u].y | (d[u].z << 8), d[u].w, v.qslot[d[u].x]) : make_int4(0, 0, 0, -1);
#pragma unroll
    for (int u = 0; u < PL_BATCH; ++u) {
      if (f0 + u * 1024 >= n_all) break;                         // uniform across the CTA
      const int4 e = ent[u];
      const unsigned keep = e.w >= 0 ? 1u : 0u;
      unsigned ik = keep;                                         // inclusive scan inside the warp
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned a = __shfl_up_sync(0xffffffffu, ik, o);
        if (lane >= o) ik += a;
      }
      if (lane == 31) s_wsum[warp] = ik;
      __syncthreads();
      if (warp == 0) {
        unsigned wk = s_wsum[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned a = __shfl_up_sync(0xffffffffu, wk, o);
          if (lane >= o) wk += a;
        }
        s_wsum[lane] = wk;                                        // inclusive over warps
      }
      __syncthreads();
      const unsigned pk = s_base + (warp ? s_wsum[warp - 1] : 0u) + ik - keep;      // exclusive position
      if (keep) { v.klist[pk] = e; atomicAdd(&s_keep[run_[u]], 1); }
      __syncthreads();
      if (tid == 0) s_base += s_wsum[31];
      __syncthreads();
    }
  }
  // class runs of the kept list: tiles, items (a pair item holds two tiles) and estimated cost before each run
  if (tid == 0) {
    int ko = 0, io = 0;
    unsigned long long co = 0ull;
    for (int k = 0; k < v.NC; ++k) {
      s_koff[k] = ko; s_ioff[k] = io; s_coff[k] = co;
      const int items = pairs ? (s_keep[k] + 1) / 2 : s_keep[k];
      ko += s_keep[k]; io += items;
      co += (unsigned long long)items * ktile_cost(v.NC - k);
    }
    s_koff[v.NC] = ko; s_ioff[v.NC] = io; s_coff[v.NC] = co;
    *v.klist_count = ko;
    v.cta_start[n_cta] = io;
  }
  __syncthreads();
  const int n_items = s_ioff[v.NC];
  const unsigned long long total = s_coff[v.NC];
  if (pairs) {
    for (int i = tid; i < n_items; i += blockDim.x) {
      int k = 0;
      while (i >= s_ioff[k + 1]) ++k;
      const int t0 = s_koff[k] + 2 * (i - s_ioff[k]);
      const int4 e0 = v.klist[t0];
      // a run of odd length ends with a filler: the same tile again, flagged so that its scores are dropped
      v.kpairs[2 * i] = e0;
      v.kpairs[2 * i + 1] = t0 + 1 < s_koff[k + 1] ? v.klist[t0 + 1] : make_int4(e0.x, e0.y | 0x80, e0.z, e0.w);
    }
  }
  // cut points: piece b starts at the item whose cost interval holds b / n_cta of the total (64-bit arithmetic; inside
  // a run every item costs the same, so the item follows from a division)
  for (int b = tid; b < n_cta; b += blockDim.x) {
    int start = 0;
    if (n_items > 0 && total > 0ull) {
      const unsigned long long key = (unsigned long long)b * total / (unsigned long long)n_cta;
      int k = 0;
      while (k + 1 < v.NC && s_coff[k + 1] <= key) ++k;
      const unsigned long long within = (key - s_coff[k]) / ktile_cost(v.NC - k);
      const int cap = s_ioff[k + 1] - s_ioff[k];
      start = s_ioff[k] + (int)(within < (unsigned long long)cap ? within : (unsigned long long)cap);
    }
    v.cta_start[b] = start;
  }
}

// ------------------------------------------------------------------------ V accumulate
constexpr int VA_GROUP = 4;                                        // panels of a tile that share one read of the probabilities
constexpr int VA_STAGES = 2 * VA_GROUP + 1;                       // the group being read + the group being refilled + one

// One CTA per (query slot, split, head group of <= 32 heads).  A warp owns one 16-head row tile (warp / 8) and the
// (warp % 8)-th group of 8 columns of every 64-column panel, so every rank class keeps all warps busy and a thread
// carries 64 accumulators.  NWG = 1 (up to 16 heads, 8 warps) or 2 (up to 32 heads, 16 warps).
// Panels arrive through a ring of cp.async stages; a tile's panels are consumed in groups of up to VA_GROUP that
// share one ldmatrix read of the tile's probability fragments (shared-memory reads bound this kernel).
template <bool BF16, int NWG>
__global__ void __launch_bounds__(256 * NWG, 1)
vacc_kernel(DevView v, int layer, const int* __restrict__ seq_ids, int n_splits) {
  constexpr int NT = 256 * NWG;                                    // threads
  constexpr int TPT = 2 * NWG;                                     // threads per token in the probability phase, 8 heads each
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* sV = smem;                                        // [STAGES][128 tokens][128 B]
  // [2][32 heads][256 B]; bf16 keeps a second pair of buffers for the low parts of the weights (see below)
  unsigned char* sP = smem + VA_STAGES * 16384;
  constexpr int P_BYTES = (BF16 ? 4 : 2) * 8192;
  float* sM = reinterpret_cast<float*>(sP + P_BYTES);              // [32] reference max per head

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mt = warp >> 3, cw = warp & 7;                         // row tile, column group
  const int Hq = v.Hq;
  const int qs = blockIdx.x / n_splits, split = blockIdx.x - qs * n_splits;
  const int h0 = blockIdx.y * 32, nh = min(32, Hq - h0);
  const int seq = seq_ids[qs];
  if (seq < 0 || seq >= v.S) return;
  const int n_tiles = v.svc(layer)[seq];
  const int* list = v.svt(layer) + (size_t)seq * v.TPS;
  const int4* desc = v.desc(layer, 1);
  const int* aux = v.aux(layer, 1);

  for (int i = tid; i < P_BYTES / 4; i += NT) reinterpret_cast<unsigned*>(sP)[i] = 0u;
  if (tid < 32) {
    // a query that sees no token (chunked prefill, every cached position after its own) has no maximum: weights stay 0
    const float m = tid < nh ? dec_ordered(v.seqmax[qs * Hq + h0 + tid]) : 0.f;
    sM[tid] = m == -INFINITY ? 0.f : m;
  }
  // Descriptors of this split's tiles (the k-th is list[split + k * n_splits]) are kept in a ring of 64 in
  // shared memory, refilled 16 at a time well ahead of both cursors, so neither the copy cursor nor the
  // consumer waits for the two dependent global reads list -> descriptor.
  __shared__ int4 s_desc[64];
  __shared__ int s_tile[64];
  const int n_mine = n_tiles > split ? (n_tiles - split + n_splits - 1) / n_splits : 0;
  auto refill = [&](int k_lo) {                                    // entries k_lo .. k_lo + 15, one thread each
    if (tid < 16 && k_lo + tid < n_mine) {
      const int t = list[split + (k_lo + tid) * n_splits];
      s_tile[(k_lo + tid) & 63] = t;
      s_desc[(k_lo + tid) & 63] = desc[t];
    }
  };
  if (tid < 48 && tid < n_mine) {                                  // initial fill: entries 0 .. 47
    const int t = list[split + tid * n_splits];
    s_tile[tid] = t;
    s_desc[tid] = desc[t];
  }
  __syncthreads();

  float acc[TWKV_MAX_CLASSES][4];
  float accl[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int p = 0; p < TWKV_MAX_CLASSES; ++p) { acc[p][0] = acc[p][1] = acc[p][2] = acc[p][3] = 0.f; }

  // producer cursor over (tile, panel) jobs of this split
  int p_k = 0, p_j = 0, p_cls = 0, p_base = 0, p_n = 0;
  auto p_load_desc = [&]() {
    if (p_k < n_mine) { const int4 d = s_desc[p_k & 63]; p_cls = d.y; p_base = d.w; }
  };
  p_load_desc();
  // this thread's 16-byte chunks of a panel: rows tid / 8 + i * NT / 8 (same row % 8, so one swizzle term), chunk tid % 8
  const unsigned cp_src_off = (unsigned)tid * 16u;
  const unsigned cp_dst_off = smem_u32(sV) + (unsigned)(tid >> 3) * 128u + ((((unsigned)tid & 7u) ^ ((unsigned)(tid >> 3) & 7u)) << 4);
  unsigned p_stage_off = 0;                                         // byte offset of the ring stage the next copy fills
  auto issue = [&]() {
    if (p_k < n_mine) {
      const unsigned char* src = v.blocks + (size_t)(p_base + p_j) * BLOCK_BYTES + cp_src_off;
      const unsigned dst = cp_dst_off + p_stage_off;
#pragma unroll
      for (int i = 0; i < 1024 / NT; ++i) cp_async16(dst + i * (NT * 16), src + i * (NT * 16));
      ++p_n;
      p_stage_off = p_stage_off == (VA_STAGES - 1) * 16384u ? 0u : p_stage_off + 16384u;
      if (++p_j == p_cls) { p_j = 0; ++p_k; p_load_desc(); }
    }
    cp_async_commit();
  };
  for (int i = 0; i < VA_STAGES - 1; ++i) issue();

  const unsigned ones = BF16 ? 0x3f803f80u : 0x3c003c00u;
  int c_n = 0, pbuf = 0;
  unsigned c_stage_off = 0;                                         // byte offset of the ring stage the next panel is read from
  int g_prev = 0;                                                   // panels of the previous group: their stages are refilled next
  // per-lane fragment addresses, fixed for the kernel.  B (V panel, transposed loads): lanes 0-15 address the 16 token
  // rows of k-step 2 i, lanes 16-31 those of k-step 2 i + 1, so one x4 load brings two k-steps; the swizzle term only
  // depends on row % 8 = lane % 8.  A (probabilities): row and 16-byte chunk of the lane's 8 x 8 matrix per k-step.
  const unsigned frag_b_off = smem_u32(sV) + (unsigned)((lane & 15) + (lane >> 4) * 16) * 128u + (((unsigned)cw ^ ((unsigned)lane & 7u)) << 4);
  unsigned frag_a_off[8];
  {
    const int mat = lane >> 3, rin = lane & 7, row = mt * 16 + rin + (mat & 1) * 8;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) frag_a_off[ks] = smem_u32(sP) + (unsigned)row * 256u + ((unsigned)((ks * 2 + (mat >> 1)) ^ rin) << 4);
  }
  // Scores of a tile are fetched one tile ahead (the V slot's link to its score row two tiles ahead),
  // so the gather's latency hides behind the previous tile's panels.
  const int slot = tid / TPT, part = tid % TPT;                    // TPT threads per token, 8 heads each
  float sc_next[8];
  int link_next = -1;                                              // score row of this thread's token in the tile after next (-1: none)
  auto fetch_link = [&](int k) {
    link_next = -1;
    if (k < n_mine && slot < s_desc[k & 63].z) link_next = aux[(size_t)s_tile[k & 63] * TILE + slot];
  };
  auto fetch_scores = [&]() {                                      // uses link_next
    if (link_next >= 0) {
      const float* srow = v.scores + (size_t)link_next * Hq + h0 + part * 8;
      if ((Hq & 3) == 0) {                                         // rows are 16-byte aligned: four heads per load
#pragma unroll
        for (int hh = 0; hh < 8; hh += 4) {
          if (part * 8 + hh < nh) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(srow + hh));
            sc_next[hh] = t.x; sc_next[hh + 1] = t.y; sc_next[hh + 2] = t.z; sc_next[hh + 3] = t.w;
          } else {
            sc_next[hh] = sc_next[hh + 1] = sc_next[hh + 2] = sc_next[hh + 3] = -INFINITY;
          }
        }
      } else {
#pragma unroll
        for (int hh = 0; hh < 8; ++hh) sc_next[hh] = (part * 8 + hh < nh) ? __ldg(srow + hh) : -INFINITY;
      }
    } else {
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) sc_next[hh] = -INFINITY;
    }
  };
  fetch_link(0);
  fetch_scores();
  fetch_link(1);
  for (int k = 0; k < n_mine; ++k) {
    if ((k & 15) == 0) refill(k + 48);                             // used from tile k + 16 on; many barriers in between
    const int cls = s_desc[k & 63].y;
    // probabilities of this tile's tokens: p = exp(s - max), rounded to the storage type.  No barrier is needed here:
    // the buffer was last read two tiles ago, and every warp has since passed a group barrier of the previous tile;
    // the first group barrier below publishes the new values.
    {
      unsigned char* P = sP + pbuf * 8192;
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) {
        const int h = part * 8 + hh;
        if (h < nh) {
          const float pv = __expf(sc_next[hh] - sM[h]);             // -inf for rows past the last token: weight 0
          const int chunk = slot >> 3;
          const unsigned short ph = from_f32<BF16>(pv);
          *reinterpret_cast<unsigned short*>(P + h * 256 + ((chunk ^ (h & 7)) << 4) + (slot & 7) * 2) = ph;
          // bf16 keeps 8 bits of a weight: with few tokens per sequence that rounding alone reaches 1e-3 of the output,
          // so the remainder goes into a second operand (16 bits in all, like an f16 weight's 11 where it matters)
          if constexpr (BF16)
            *reinterpret_cast<unsigned short*>(P + 16384 + h * 256 + ((chunk ^ (h & 7)) << 4) + (slot & 7) * 2) =
                from_f32<true>(pv - to_f32<true>(ph));
        }
      }
    }
    fetch_scores();                                                // next tile's scores (link fetched one tile ago)
    fetch_link(k + 2);
    // The tile's panels are taken in groups of up to VA_GROUP: the probability fragments of a k-step are read from
    // shared memory once per group instead of once per panel (they were two thirds of the shared-memory reads, which
    // bound this kernel).  The stages the previous group occupied are refilled while this one is read.
    for (int j0 = 0; j0 < cls; j0 += VA_GROUP) {
      const int g = min(VA_GROUP, cls - j0);
      // copies still allowed in flight once this group's panels have landed: everything issued after them
      switch (VA_STAGES - 1 - g_prev - g) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        default: cp_async_wait<6>(); break;
      }
      __syncthreads();
      for (int i = 0; i < g_prev; ++i) issue();
      g_prev = g;
      unsigned vAddr[VA_GROUP];
#pragma unroll
      for (int jj = 0; jj < VA_GROUP; ++jj) {
        unsigned o = c_stage_off + jj * 16384u;
        if (o >= VA_STAGES * 16384u) o -= VA_STAGES * 16384u;
        vAddr[jj] = frag_b_off + o;
      }
      c_stage_off += (unsigned)g * 16384u;
      if (c_stage_off >= VA_STAGES * 16384u) c_stage_off -= VA_STAGES * 16384u;
      c_n += g;
      const unsigned pOff = (unsigned)pbuf * 8192u;
      // first panel and group size select the accumulators at compile time so they stay in registers
      auto do_group = [&](auto J0, auto G) {
        constexpr int jbase = decltype(J0)::value, gn = decltype(G)::value;
#pragma unroll
        for (int k2 = 0; k2 < 4; ++k2) {                           // two k-steps (32 tokens) per iteration
          unsigned a0[4], a1[4];
          [[maybe_unused]] unsigned l0[4], l1[4];
          ldsm_x4(a0, frag_a_off[2 * k2] + pOff);
          ldsm_x4(a1, frag_a_off[2 * k2 + 1] + pOff);
          if constexpr (BF16) {
            ldsm_x4(l0, frag_a_off[2 * k2] + pOff + 16384u);
            ldsm_x4(l1, frag_a_off[2 * k2 + 1] + pOff + 16384u);
          }
#pragma unroll
          for (int jj = 0; jj < gn; ++jj) {
            if (jbase + jj < TWKV_MAX_CLASSES) {
              unsigned b[4];
              ldsm_x4_t(b, vAddr[jj] + k2 * 4096);
              mma16816<BF16>(acc[jbase + jj < TWKV_MAX_CLASSES ? jbase + jj : 0], a0, b[0], b[1]);
              mma16816<BF16>(acc[jbase + jj < TWKV_MAX_CLASSES ? jbase + jj : 0], a1, b[2], b[3]);
              if constexpr (BF16) {
                mma16816<BF16>(acc[jbase + jj < TWKV_MAX_CLASSES ? jbase + jj : 0], l0, b[0], b[1]);
                mma16816<BF16>(acc[jbase + jj < TWKV_MAX_CLASSES ? jbase + jj : 0], l1, b[2], b[3]);
              }
            }
          }
          if (jbase == 0 && cw == 0) {
            mma16816<BF16>(accl, a0, ones, ones); mma16816<BF16>(accl, a1, ones, ones);
            if constexpr (BF16) { mma16816<BF16>(accl, l0, ones, ones); mma16816<BF16>(accl, l1, ones, ones); }
          }
        }
      };
      auto by_size = [&](auto J0) {
        switch (g) {
          case 1: do_group(J0, std::integral_constant<int, 1>{}); break;
          case 2: do_group(J0, std::integral_constant<int, 2>{}); break;
          case 3: do_group(J0, std::integral_constant<int, 3>{}); break;
          default: do_group(J0, std::integral_constant<int, 4>{}); break;
        }
      };
      switch (j0) {
        case 0: by_size(std::integral_constant<int, 0>{}); break;
        case 4: by_size(std::integral_constant<int, 4>{}); break;
        case 8: by_size(std::integral_constant<int, 8>{}); break;
        default: by_size(std::integral_constant<int, 12>{}); break;
      }
    }
    pbuf ^= 1;
  }
  cp_async_wait<0>();

  // partial results of this split
  const size_t pidx = (size_t)qs * n_splits + split;
  float* pa = v.part_acc + pidx * Hq * v.d_kv;
  const int r0 = mt * 16 + (lane >> 2), r1 = r0 + 8;
#pragma unroll
  for (int pj = 0; pj < TWKV_MAX_CLASSES; ++pj) {
    if (pj < v.NC) {
      const int col = pj * PANEL + cw * 8 + (lane & 3) * 2;
      if (r0 < nh) *reinterpret_cast<float2*>(pa + (size_t)(h0 + r0) * v.d_kv + col) = make_float2(acc[pj][0], acc[pj][1]);
      if (r1 < nh) *reinterpret_cast<float2*>(pa + (size_t)(h0 + r1) * v.d_kv + col) = make_float2(acc[pj][2], acc[pj][3]);
    }
  }
  if (cw == 0 && (lane & 3) == 0) {
    if (r0 < nh) v.part_l[pidx * Hq + h0 + r0] = accl[0];
    if (r1 < nh) v.part_l[pidx * Hq + h0 + r1] = accl[2];
  }
}

// -------------------------------------------------------------- merge + V projection
// One CTA per (query slot, KV head g): sums the splits, normalises, and projects the REP heads
// of the group through U_V^-1[:, g*128 .. g*128+127].  512 threads: thread = (pair of output
// columns, one eighth of the spectral index range), several rows of U_V^-1 in flight per thread.
constexpr int MG_THREADS = 512;
constexpr int MG_JGROUPS = MG_THREADS / 64;

template <bool BF16>
__global__ void __launch_bounds__(MG_THREADS)
merge_kernel(DevView v, const unsigned short* __restrict__ Uinv_v, int n_splits, int hp, int ns, int n_seq, void* __restrict__ out) {
  extern __shared__ float sAcc[];                    // [rows][d_kv] normalised spectral accumulators, then [MG_JGROUPS][rows][128]
  __shared__ float sInvL[8];
  // blockIdx.y = KV head g and which hp of its query heads (hp divides the group size; small batches use hp < group
  // size so that the grid still fills the device); blockIdx.x = ns query slots that share the reads of U_V^-1 (large
  // batches).  A row of this CTA is (slot, head): at most 8 rows.
  const int qs0 = blockIdx.x * ns, parts = v.rep / hp, g = blockIdx.y / parts, tid = threadIdx.x;
  const int Hq = v.Hq, d_kv = v.d_kv;
  const int REP = min(ns, n_seq - qs0) * hp;                    // rows
  const int head0 = g * v.rep + (blockIdx.y % parts) * hp;      // first query head of this CTA
  if (tid < REP) {
    const int qs = qs0 + tid / hp, head = head0 + tid % hp;
    float l = 0.f;
    for (int s = 0; s < n_splits; ++s) l += v.part_l[((size_t)qs * n_splits + s) * Hq + head];
    sInvL[tid] = l > 0.f ? 1.f / l : 0.f;
  }
  __syncthreads();
  // split sums in split order; four elements per thread at a time so that four reads per split are in flight
  for (int i0 = tid; i0 < REP * d_kv; i0 += 4 * MG_THREADS) {
    const float* p[4];
    float a[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = min(i0 + u * MG_THREADS, REP * d_kv - 1), hh = i / d_kv, j = i - hh * d_kv;
      p[u] = v.part_acc + (((size_t)(qs0 + hh / hp) * n_splits) * Hq + head0 + hh % hp) * d_kv + j;
    }
    for (int s = 0; s < n_splits; ++s) {
#pragma unroll
      for (int u = 0; u < 4; ++u) a[u] += __ldg(p[u] + (size_t)s * Hq * d_kv);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * MG_THREADS;
      if (i < REP * d_kv) sAcc[i] = a[u] * sInvL[i / d_kv];
    }
  }
  __syncthreads();
  const int dp = tid & 63, jg = tid >> 6;
  const int jn = d_kv / MG_JGROUPS, j0 = jg * jn;
  float o[8][2];
#pragma unroll
  for (int h = 0; h < 8; ++h) { o[h][0] = 0.f; o[h][1] = 0.f; }
  const unsigned* ucol = reinterpret_cast<const unsigned*>(Uinv_v + g * HEAD_DIM) + dp;    // two 16-bit columns per load
  for (int jb = 0; jb < jn; jb += 16) {                // jn is a multiple of 16 (d_kv a multiple of 128)
    unsigned u[16];
#pragma unroll
    for (int t = 0; t < 16; ++t) u[t] = __ldg(ucol + (size_t)(j0 + jb + t) * (d_kv / 2));
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      const float u0 = to_f32<BF16>((unsigned short)(u[t] & 0xffffu)), u1 = to_f32<BF16>((unsigned short)(u[t] >> 16));
#pragma unroll
      for (int h = 0; h < 8; ++h)
        if (h < REP) {
          const float a = sAcc[h * d_kv + j0 + jb + t];
          o[h][0] += a * u0;
          o[h][1] += a * u1;
        }
    }
  }
  __syncthreads();
  float* red = sAcc;                                 // reuse: [MG_JGROUPS][REP][128]
#pragma unroll
  for (int h = 0; h < 8; ++h)
    if (h < REP) *reinterpret_cast<float2*>(red + (jg * REP + h) * 128 + 2 * dp) = make_float2(o[h][0], o[h][1]);
  __syncthreads();
  for (int i = tid; i < REP * 128; i += MG_THREADS) {
    float val = 0.f;
#pragma unroll
    for (int k = 0; k < MG_JGROUPS; ++k) val += red[k * REP * 128 + i];        // fixed order
    const int h = i >> 7, dc = i & 127;
    const int oslot = qs0 + h / hp;
    const size_t oi = ((size_t)(v.qmap ? v.qmap[oslot] : oslot) * Hq + head0 + h % hp) * HEAD_DIM + dc;
    if (v.out_dtype == TWKV_F32) reinterpret_cast<float*>(out)[oi] = val;
    else if (v.out_dtype == TWKV_BF16) reinterpret_cast<unsigned short*>(out)[oi] = from_f32<true>(val);
    else reinterpret_cast<unsigned short*>(out)[oi] = from_f32<false>(val);
  }
}

// ------------------------------------------------------------------------- host side
cudaError_t launch_kscore_tc(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                             const void* q, int n_pieces, bool pairs, cudaStream_t st);

template <bool BF16>
static cudaError_t launch_decode_t(const DevView& v, int layer, const LayerParams& lp, const void* q, const int* seq_ids,
                                   int n_seq, void* out, int n_splits, int sm_count, const TcMaps* maps, bool pairs, cudaStream_t st) {
  // the K-score kernel's work is cut into one piece per persistent CTA, or per CTA pair
  const int n_pieces = pairs ? kscore_max_pairs(sm_count) : sm_count;
  { ProfScope ps(TWKV_K_PLAN, st); plan_kernel<<<1, 1024, 0, st>>>(v, layer, seq_ids, n_seq, n_pieces, pairs ? 1 : 0); }
  {
    cudaError_t e = launch_kscore_tc(v, layer, maps->blocks, maps->uinvT_k, q, n_pieces, pairs, st);
    if (e != cudaSuccess) return e;
  }
  const size_t va_smem = VA_STAGES * 16384 + (BF16 ? 4 : 2) * 8192 + 32 * 4;
  const dim3 vgrid(n_seq * n_splits, (v.Hq + 31) / 32);
  if (v.Hq <= 16) {
    cudaFuncSetAttribute(vacc_kernel<BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)va_smem);
    ProfScope ps(TWKV_K_VACC, st);
    vacc_kernel<BF16, 1><<<vgrid, 256, va_smem, st>>>(v, layer, seq_ids, n_splits);
  } else {
    cudaFuncSetAttribute(vacc_kernel<BF16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)va_smem);
    ProfScope ps(TWKV_K_VACC, st);
    vacc_kernel<BF16, 2><<<vgrid, 512, va_smem, st>>>(v, layer, seq_ids, n_splits);
  }
  // query heads per merge CTA: the whole group when the batch fills the device, fewer (a divisor) for small batches;
  // query slots per CTA: more than one (they share the reads of U_V^-1) while the grid still fills most of the device
  int hp = v.rep;
  while (hp % 2 == 0 && 2 * n_seq * v.Hkv * (v.rep / hp) < sm_count) hp /= 2;
  int ns = 1;
  while (2 * ns * hp <= 8 && 4 * (n_seq * v.Hkv * (v.rep / hp) / (2 * ns)) >= 3 * sm_count) ns *= 2;
  const size_t mg_a = (size_t)ns * hp * v.d_kv * 4, mg_b = (size_t)MG_JGROUPS * ns * hp * 128 * 4;
  const size_t mg_smem = mg_a > mg_b ? mg_a : mg_b;
  {
    ProfScope ps(TWKV_K_MERGE, st);
    merge_kernel<BF16><<<dim3((n_seq + ns - 1) / ns, v.Hkv * (v.rep / hp)), MG_THREADS, mg_smem, st>>>(
        v, reinterpret_cast<const unsigned short*>(lp.Uinv_v), n_splits, hp, ns, n_seq, out);
  }
  count_launch(4);
  return cudaGetLastError();
}

cudaError_t launch_decode(const DevView& v, int layer, const LayerParams& lp, const void* q, const int* seq_ids,
                          int n_seq, void* out, int num_splits, int sm_count, const TcMaps* maps, bool pairs, cudaStream_t st) {
  if (n_seq <= 0) return cudaSuccess;
  return v.dtype == TWKV_BF16 ? launch_decode_t<true>(v, layer, lp, q, seq_ids, n_seq, out, num_splits, sm_count, maps, pairs, st)
                              : launch_decode_t<false>(v, layer, lp, q, seq_ids, n_seq, out, num_splits, sm_count, maps, pairs, st);
}

}  // namespace twkv
