// Decode attention over the mixed-rank cache (Eq. 3, reshape to heads, RoPE, softmax attention).
//
//   plan_kernel    sequence id -> query slot map, running-max reset
//   kscore_kernel  per K tile: Kbar = X^_K U_K^-1 (tensor cores), RoPE by stored position,
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
__global__ void plan_kernel(DevView v, const int* __restrict__ seq_ids, int n_seq) {
  for (int s = threadIdx.x; s < v.S; s += blockDim.x) v.qslot[s] = -1;
  __syncthreads();
  for (int i = threadIdx.x; i < n_seq; i += blockDim.x) {
    const int s = seq_ids[i];
    if (s < 0 || s >= v.S) set_status(v, TWKV_ERR_INVALID_ARG);
    else v.qslot[s] = i;
  }
  for (int i = threadIdx.x; i < n_seq * v.Hq; i += blockDim.x) v.seqmax[i] = 0u;
  __syncthreads();
  for (int i = threadIdx.x; i < n_seq; i += blockDim.x) {
    const int s = seq_ids[i];
    if (s >= 0 && s < v.S && v.qslot[s] != i) set_status(v, TWKV_ERR_INVALID_ARG);   // duplicate id
  }
}

// ---------------------------------------------------------------------------- K scores
constexpr int KS_STAGES = 3;
constexpr int KS_THREADS = 256;

template <bool BF16, int REP>
__global__ void __launch_bounds__(KS_THREADS, 1)
kscore_kernel(DevView v, int layer, const unsigned short* __restrict__ Uinv, const unsigned short* __restrict__ q) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* sA = smem;                                   // [STAGES][128 rows][128 B]
  unsigned char* sB = smem + KS_STAGES * 16384;               // [STAGES][64 k][256 B]
  float* sQ = reinterpret_cast<float*>(smem + 2 * KS_STAGES * 16384);   // [Hq][128], pre-scaled
  float* sS = sQ + v.Hq * HEAD_DIM;                           // [128][Hq]
  __shared__ int s_cls_cnt[TWKV_MAX_CLASSES];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hq = v.Hq, d_kv = v.d_kv, Hkv = v.Hkv;
  const int* kcc = v.kcc(layer);
  if (tid < TWKV_MAX_CLASSES) s_cls_cnt[tid] = tid < v.NC ? kcc[tid] : 0;
  __syncthreads();
  int total = 0;
  for (int c = 0; c < v.NC; ++c) total += s_cls_cnt[c];
  const int4* desc = v.desc(layer, 0);
  const int* aux = v.aux(layer, 0);
  const int* kct = v.kct(layer);

  for (int w = blockIdx.x; w < total; w += gridDim.x) {
    // work items are ordered from the widest class to the narrowest
    int cls = v.NC, idx = w;
    while (idx >= s_cls_cnt[cls - 1]) { idx -= s_cls_cnt[cls - 1]; --cls; }
    const int tile = kct[(size_t)(cls - 1) * v.NT + idx];
    const int4 dsc = desc[tile];
    const int qs = v.qslot[dsc.x];
    if (qs < 0) continue;
    const int n_valid = dsc.z, base = dsc.w;
    __syncthreads();                                          // previous tile's smem is free
    for (int i = tid; i < Hq * HEAD_DIM; i += KS_THREADS)
      sQ[i] = to_f32<BF16>(q[(size_t)qs * Hq * HEAD_DIM + i]) * v.sm_scale;

    // cos / sin of this thread's two rows and sixteen frequencies
    const int row0 = warp * 16 + (lane >> 2), row1 = row0 + 8;
    float cs0[16], sn0[16], cs1[16], sn1[16];
    {
      const int p0 = aux[(size_t)tile * TILE + row0], p1 = aux[(size_t)tile * TILE + row1];
      const float2* h0 = v.rope_hi + (size_t)((p0 >> 9) & (ROPE_HI - 1)) * 64;
      const float2* l0 = v.rope_lo + (size_t)(p0 & (ROPE_LO - 1)) * 64;
      const float2* h1 = v.rope_hi + (size_t)((p1 >> 9) & (ROPE_HI - 1)) * 64;
      const float2* l1 = v.rope_lo + (size_t)(p1 & (ROPE_LO - 1)) * 64;
#pragma unroll
      for (int f = 0; f < 16; ++f) {
        const int fi = (f >> 1) * 8 + (lane & 3) * 2 + (f & 1);
        float2 a = h0[fi], b = l0[fi];
        cs0[f] = a.x * b.x - a.y * b.y; sn0[f] = a.y * b.x + a.x * b.y;
        a = h1[fi]; b = l1[fi];
        cs1[f] = a.x * b.x - a.y * b.y; sn1[f] = a.y * b.x + a.x * b.y;
      }
    }

    const int iters = Hkv * cls;
    auto issue = [&](int it) {
      if (it < iters) {
        const int g = it / cls, j = it - g * cls, st = it % KS_STAGES;
        const unsigned char* srcA = v.blocks + (size_t)(base + j) * BLOCK_BYTES;
        const unsigned dA = smem_u32(sA + st * 16384);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = tid + i * KS_THREADS, row = c >> 3, ch = c & 7;
          cp_async16(dA + row * 128 + ((ch ^ (row & 7)) << 4), srcA + row * 128 + ch * 16);
        }
        const unsigned char* srcB = reinterpret_cast<const unsigned char*>(Uinv) + ((size_t)(j * PANEL) * d_kv + g * HEAD_DIM) * 2;
        const unsigned dB = smem_u32(sB + st * 16384);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = tid + i * KS_THREADS, kr = c >> 4, ch = c & 15;
          cp_async16(dB + kr * 256 + ((ch ^ (kr & 7)) << 4), srcB + (size_t)kr * d_kv * 2 + ch * 16);
        }
      }
      cp_async_commit();
    };
    for (int it = 0; it < KS_STAGES - 1; ++it) issue(it);

    float acc[16][4];
    for (int it = 0; it < iters; ++it) {
      const int g = it / cls, j = it - g * cls, st = it % KS_STAGES;
      if (j == 0) {
#pragma unroll
        for (int n = 0; n < 16; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
      }
      cp_async_wait<KS_STAGES - 2>();
      __syncthreads();
      issue(it + KS_STAGES - 1);
      const unsigned aBase = smem_u32(sA + st * 16384), bBase = smem_u32(sB + st * 16384);
      const int mat = lane >> 3, rin = lane & 7;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        unsigned a[4];
        {
          const int row = warp * 16 + rin + (mat & 1) * 8, kc = ks * 2 + (mat >> 1);
          ldsm_x4(a, aBase + row * 128 + ((kc ^ (row & 7)) << 4));
        }
#pragma unroll
        for (int np = 0; np < 8; ++np) {
          unsigned b[4];
          const int kr = ks * 16 + rin + (mat & 1) * 8, nc = np * 2 + (mat >> 1);
          ldsm_x4_t(b, bBase + kr * 256 + ((nc ^ (kr & 7)) << 4));
          mma16816<BF16>(acc[np * 2], a, b[0], b[1]);
          mma16816<BF16>(acc[np * 2 + 1], a, b[2], b[3]);
        }
      }
      if (j == cls - 1) {
        // slab g is complete: RoPE pairs (i, i + 64) live in n-tiles (n, n + 8) of the same thread
        float s0[REP], s1[REP];
#pragma unroll
        for (int h = 0; h < REP; ++h) { s0[h] = 0.f; s1[h] = 0.f; }
#pragma unroll
        for (int n = 0; n < 8; ++n) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int f = n * 2 + e, dim = n * 8 + (lane & 3) * 2 + e;
            const float x1 = acc[n][e], x2 = acc[n + 8][e];
            const float y1 = x1 * cs0[f] - x2 * sn0[f], y2 = x2 * cs0[f] + x1 * sn0[f];
            const float u1 = acc[n][2 + e], u2 = acc[n + 8][2 + e];
            const float z1 = u1 * cs1[f] - u2 * sn1[f], z2 = u2 * cs1[f] + u1 * sn1[f];
#pragma unroll
            for (int h = 0; h < REP; ++h) {
              const float qa = sQ[(g * REP + h) * HEAD_DIM + dim], qb = sQ[(g * REP + h) * HEAD_DIM + dim + 64];
              s0[h] += y1 * qa + y2 * qb;
              s1[h] += z1 * qa + z2 * qb;
            }
          }
        }
#pragma unroll
        for (int h = 0; h < REP; ++h) {
          s0[h] += __shfl_xor_sync(0xffffffffu, s0[h], 1); s0[h] += __shfl_xor_sync(0xffffffffu, s0[h], 2);
          s1[h] += __shfl_xor_sync(0xffffffffu, s1[h], 1); s1[h] += __shfl_xor_sync(0xffffffffu, s1[h], 2);
          if ((lane & 3) == 0) {
            sS[row0 * Hq + g * REP + h] = s0[h];
            sS[row1 * Hq + g * REP + h] = s1[h];
          }
        }
      }
    }
    cp_async_wait<0>();
    __syncthreads();
    float* out = v.scores + (size_t)tile * TILE * Hq;
    for (int i = tid; i < TILE * Hq; i += KS_THREADS) out[i] = (i / Hq < n_valid) ? sS[i] : -INFINITY;
    if (tid < Hq) {
      float m = -INFINITY;
      for (int r = 0; r < n_valid; ++r) m = fmaxf(m, sS[r * Hq + tid]);
      atomicMax(&v.seqmax[qs * Hq + tid], enc_ordered(m));
    }
  }
}

// ------------------------------------------------------------------------ V accumulate
constexpr int VA_STAGES = 6;
constexpr int VA_THREADS = 256;

// One CTA per (query slot, split, head group of <= 32 heads).  Warp w owns the w-th group of 8
// columns of every 64-column panel, so every rank class keeps all eight warps busy.
template <bool BF16, int MTW>
__global__ void __launch_bounds__(VA_THREADS, 1)
vacc_kernel(DevView v, int layer, const int* __restrict__ seq_ids, int n_splits) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* sV = smem;                                        // [STAGES][128 tokens][128 B]
  unsigned char* sP = smem + VA_STAGES * 16384;                    // [2][32 heads][256 B]
  float* sM = reinterpret_cast<float*>(sP + 2 * 8192);             // [32] reference max per head

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hq = v.Hq;
  const int qs = blockIdx.x / n_splits, split = blockIdx.x - qs * n_splits;
  const int h0 = blockIdx.y * 32, nh = min(32, Hq - h0);
  const int seq = seq_ids[qs];
  if (seq < 0 || seq >= v.S) return;
  const int n_tiles = v.svc(layer)[seq];
  const int* list = v.svt(layer) + (size_t)seq * v.TPS;
  const int4* desc = v.desc(layer, 1);
  const int* aux = v.aux(layer, 1);

  for (int i = tid; i < 2 * 8192 / 4; i += VA_THREADS) reinterpret_cast<unsigned*>(sP)[i] = 0u;
  if (tid < 32) sM[tid] = tid < nh ? dec_ordered(v.seqmax[qs * Hq + h0 + tid]) : 0.f;

  float acc[TWKV_MAX_CLASSES][MTW][4];
  float accl[MTW][4];
#pragma unroll
  for (int p = 0; p < TWKV_MAX_CLASSES; ++p)
#pragma unroll
    for (int m = 0; m < MTW; ++m) { acc[p][m][0] = acc[p][m][1] = acc[p][m][2] = acc[p][m][3] = 0.f; }
#pragma unroll
  for (int m = 0; m < MTW; ++m) { accl[m][0] = accl[m][1] = accl[m][2] = accl[m][3] = 0.f; }

  // producer cursor over (tile, panel) jobs of this split
  int p_ti = split, p_j = 0, p_cls = 0, p_base = 0, p_n = 0;
  auto p_load_desc = [&]() {
    if (p_ti < n_tiles) { const int4 d = desc[list[p_ti]]; p_cls = d.y; p_base = d.w; }
  };
  p_load_desc();
  auto issue = [&]() {
    if (p_ti < n_tiles) {
      const unsigned char* src = v.blocks + (size_t)(p_base + p_j) * BLOCK_BYTES;
      const unsigned dst = smem_u32(sV + (p_n % VA_STAGES) * 16384);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = tid + i * VA_THREADS, row = c >> 3, ch = c & 7;
        cp_async16(dst + row * 128 + ((ch ^ (row & 7)) << 4), src + row * 128 + ch * 16);
      }
      ++p_n;
      if (++p_j == p_cls) { p_j = 0; p_ti += n_splits; p_load_desc(); }
    }
    cp_async_commit();
  };
  for (int i = 0; i < VA_STAGES - 1; ++i) issue();

  const unsigned ones = BF16 ? 0x3f803f80u : 0x3c003c00u;
  int c_n = 0, pbuf = 0;
  for (int ti = split; ti < n_tiles; ti += n_splits) {
    const int tile = list[ti];
    const int4 dsc = desc[tile];
    const int cls = dsc.y, n_valid = dsc.z;
    // probabilities of this tile's tokens: p = exp(s - max), rounded to the storage type
    __syncthreads();
    {
      unsigned char* P = sP + pbuf * 8192;
      const int slot = tid >> 1, part = tid & 1;                   // two threads per token, 16 heads each
      const bool ok = slot < n_valid;
      const int link = ok ? aux[(size_t)tile * TILE + slot] : 0;
      const float* srow = v.scores + (size_t)link * Hq + h0;
#pragma unroll
      for (int hh = 0; hh < 16; ++hh) {
        const int h = part * 16 + hh;
        if (h < nh) {
          const float pv = ok ? __expf(srow[h] - sM[h]) : 0.f;
          const int chunk = slot >> 3;
          *reinterpret_cast<unsigned short*>(P + h * 256 + ((chunk ^ (h & 7)) << 4) + (slot & 7) * 2) = from_f32<BF16>(pv);
        }
      }
    }
    for (int j = 0; j < cls; ++j) {
      cp_async_wait<VA_STAGES - 2>();
      __syncthreads();
      issue();
      const unsigned vBase = smem_u32(sV + (c_n % VA_STAGES) * 16384);
      const unsigned pBase = smem_u32(sP + pbuf * 8192);
      ++c_n;
      // the panel index selects the accumulator at compile time so it stays in registers
      auto do_panel = [&](auto PJ) {
        constexpr int pj = decltype(PJ)::value;
        const int mat = lane >> 3, rin = lane & 7;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          unsigned b[2];
          {
            const int kr = ks * 16 + (lane & 15);
            ldsm_x2_t(b, vBase + kr * 128 + ((warp ^ (kr & 7)) << 4));
          }
#pragma unroll
          for (int m = 0; m < MTW; ++m) {
            unsigned a[4];
            const int row = m * 16 + rin + (mat & 1) * 8, kc = ks * 2 + (mat >> 1);
            ldsm_x4(a, pBase + row * 256 + ((kc ^ (row & 7)) << 4));
            mma16816<BF16>(acc[pj][m], a, b[0], b[1]);
            if (pj == 0 && warp == 0) mma16816<BF16>(accl[m], a, ones, ones);
          }
        }
      };
      switch (j) {
#define TWKV_PANEL_CASE(N) case N: do_panel(std::integral_constant<int, N>{}); break;
        TWKV_PANEL_CASE(0) TWKV_PANEL_CASE(1) TWKV_PANEL_CASE(2) TWKV_PANEL_CASE(3)
        TWKV_PANEL_CASE(4) TWKV_PANEL_CASE(5) TWKV_PANEL_CASE(6) TWKV_PANEL_CASE(7)
        TWKV_PANEL_CASE(8) TWKV_PANEL_CASE(9) TWKV_PANEL_CASE(10) TWKV_PANEL_CASE(11)
        TWKV_PANEL_CASE(12) TWKV_PANEL_CASE(13) TWKV_PANEL_CASE(14) TWKV_PANEL_CASE(15)
#undef TWKV_PANEL_CASE
        default: break;
      }
    }
    pbuf ^= 1;
  }
  cp_async_wait<0>();

  // partial results of this split
  const size_t pidx = (size_t)qs * n_splits + split;
  float* pa = v.part_acc + pidx * Hq * v.d_kv;
#pragma unroll
  for (int pj = 0; pj < TWKV_MAX_CLASSES; ++pj) {
    if (pj < v.NC) {
#pragma unroll
      for (int m = 0; m < MTW; ++m) {
        const int col = pj * PANEL + warp * 8 + (lane & 3) * 2;
        const int r0 = m * 16 + (lane >> 2), r1 = r0 + 8;
        if (r0 < nh) *reinterpret_cast<float2*>(pa + (size_t)(h0 + r0) * v.d_kv + col) = make_float2(acc[pj][m][0], acc[pj][m][1]);
        if (r1 < nh) *reinterpret_cast<float2*>(pa + (size_t)(h0 + r1) * v.d_kv + col) = make_float2(acc[pj][m][2], acc[pj][m][3]);
      }
    }
  }
  if (warp == 0 && (lane & 3) == 0) {
#pragma unroll
    for (int m = 0; m < MTW; ++m) {
      const int r0 = m * 16 + (lane >> 2), r1 = r0 + 8;
      if (r0 < nh) v.part_l[pidx * Hq + h0 + r0] = accl[m][0];
      if (r1 < nh) v.part_l[pidx * Hq + h0 + r1] = accl[m][2];
    }
  }
}

// -------------------------------------------------------------- merge + V projection
// One CTA per (query slot, KV head g): sums the splits, normalises, and projects the REP heads
// of the group through U_V^-1[:, g*128 .. g*128+127].
template <bool BF16>
__global__ void __launch_bounds__(256)
merge_kernel(DevView v, const unsigned short* __restrict__ Uinv_v, int n_splits, void* __restrict__ out) {
  extern __shared__ float sAcc[];                    // [REP][d_kv] normalised spectral accumulators, then [2][REP][128]
  const int qs = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
  const int Hq = v.Hq, d_kv = v.d_kv, REP = v.rep;
  for (int i = tid; i < REP * d_kv; i += 256) {
    const int h = g * REP + i / d_kv, j = i % d_kv;
    float a = 0.f, l = 0.f;
    for (int s = 0; s < n_splits; ++s) {
      const size_t pidx = (size_t)qs * n_splits + s;
      a += v.part_acc[(pidx * Hq + h) * d_kv + j];
      l += v.part_l[pidx * Hq + h];
    }
    sAcc[i] = l > 0.f ? a / l : 0.f;
  }
  __syncthreads();
  const int dcol = tid & 127, jh = tid >> 7;         // two threads per output column, half of j each
  float o[8];
#pragma unroll
  for (int h = 0; h < 8; ++h) o[h] = 0.f;
  const int j0 = jh * (d_kv / 2), j1 = j0 + d_kv / 2;
  for (int j = j0; j < j1; ++j) {
    const float u = to_f32<BF16>(Uinv_v[(size_t)j * d_kv + g * HEAD_DIM + dcol]);
#pragma unroll
    for (int h = 0; h < 8; ++h)
      if (h < REP) o[h] += sAcc[h * d_kv + j] * u;
  }
  __syncthreads();
  float* red = sAcc;                                 // reuse: [2][REP][128]
  for (int h = 0; h < REP; ++h) red[(jh * REP + h) * 128 + dcol] = o[h];
  __syncthreads();
  for (int i = tid; i < REP * 128; i += 256) {
    const int h = i >> 7, dc = i & 127;
    const float val = red[i] + red[REP * 128 + i];
    const size_t oi = ((size_t)qs * Hq + g * REP + h) * HEAD_DIM + dc;
    if (v.out_dtype == TWKV_F32) reinterpret_cast<float*>(out)[oi] = val;
    else if (v.out_dtype == TWKV_BF16) reinterpret_cast<unsigned short*>(out)[oi] = from_f32<true>(val);
    else reinterpret_cast<unsigned short*>(out)[oi] = from_f32<false>(val);
  }
}

// ------------------------------------------------------------------------- host side
cudaError_t launch_kscore_tc(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap& map_uinvT,
                             const void* q, int sm_count, cudaStream_t st);

template <bool BF16>
static cudaError_t launch_decode_t(const DevView& v, int layer, const LayerParams& lp, const void* q, const int* seq_ids,
                                   int n_seq, void* out, int n_splits, int sm_count, const TcMaps* maps, cudaStream_t st) {
  { ProfScope ps(TWKV_K_PLAN, st); plan_kernel<<<1, 256, 0, st>>>(v, seq_ids, n_seq); }
  if (maps) {
    cudaError_t e = launch_kscore_tc(v, layer, maps->blocks, maps->uinvT_k, q, sm_count, st);
    if (e != cudaSuccess) return e;
  } else {
  const size_t ks_smem = 2 * KS_STAGES * 16384 + (size_t)v.Hq * HEAD_DIM * 4 + (size_t)TILE * v.Hq * 4;
  const unsigned short* U = reinterpret_cast<const unsigned short*>(lp.Uinv_k);
  const unsigned short* qq = reinterpret_cast<const unsigned short*>(q);
#define TWKV_KS(REP)                                                                                              \
  {                                                                                                               \
    cudaFuncSetAttribute(kscore_kernel<BF16, REP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ks_smem);    \
    ProfScope ps(TWKV_K_KSCORE, st);                                                                              \
    kscore_kernel<BF16, REP><<<sm_count, KS_THREADS, ks_smem, st>>>(v, layer, U, qq);                             \
  }
  switch (v.rep) {
    case 1: TWKV_KS(1) break;
    case 2: TWKV_KS(2) break;
    case 4: TWKV_KS(4) break;
    default: TWKV_KS(8) break;
  }
#undef TWKV_KS
  }
  const size_t va_smem = VA_STAGES * 16384 + 2 * 8192 + 32 * 4;
  const dim3 vgrid(n_seq * n_splits, (v.Hq + 31) / 32);
  if (v.Hq <= 16) {
    cudaFuncSetAttribute(vacc_kernel<BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)va_smem);
    ProfScope ps(TWKV_K_VACC, st);
    vacc_kernel<BF16, 1><<<vgrid, VA_THREADS, va_smem, st>>>(v, layer, seq_ids, n_splits);
  } else {
    cudaFuncSetAttribute(vacc_kernel<BF16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)va_smem);
    ProfScope ps(TWKV_K_VACC, st);
    vacc_kernel<BF16, 2><<<vgrid, VA_THREADS, va_smem, st>>>(v, layer, seq_ids, n_splits);
  }
  const size_t mg_smem = (size_t)v.rep * v.d_kv * 4;
  {
    ProfScope ps(TWKV_K_MERGE, st);
    merge_kernel<BF16><<<dim3(n_seq, v.Hkv), 256, mg_smem, st>>>(v, reinterpret_cast<const unsigned short*>(lp.Uinv_v), n_splits, out);
  }
  count_launch(4);
  return cudaGetLastError();
}

cudaError_t launch_decode(const DevView& v, int layer, const LayerParams& lp, const void* q, const int* seq_ids,
                          int n_seq, void* out, int num_splits, int sm_count, const TcMaps* maps, cudaStream_t st) {
  if (n_seq <= 0) return cudaSuccess;
  return v.dtype == TWKV_BF16 ? launch_decode_t<true>(v, layer, lp, q, seq_ids, n_seq, out, num_splits, sm_count, maps, st)
                              : launch_decode_t<false>(v, layer, lp, q, seq_ids, n_seq, out, num_splits, sm_count, maps, st);
}

}  // namespace twkv
