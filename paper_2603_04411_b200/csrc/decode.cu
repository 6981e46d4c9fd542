// Decode attention over the mixed-rank cache (Eq. 3, reshape to heads, RoPE, softmax attention).
//
//   plan_kernel    sequence id -> query slot map, running-max reset, K-tile work list; cut points of every
//                  sequence's V tiles into the splits of the V pass; K slot -> V slot links of the sequences' tokens
//   kscore_tc_kernel (kscore_tc.cu)  per K tile: Kbar = X^_K U_K^-1, RoPE by stored position,
//                  s = q . Kbar * scale for the GQA group, scores to scratch, per-sequence max
//   vacc_tc_kernel (vacc_tc.cu)  per (sequence, split): p = exp(s - max), acc += p^T X^_V in spectral
//                  space (tcgen05), l = sum p
//   merge_kernel   sum of the splits, out_h = (acc_h / l_h) U_V^-1[:, head slice]
//
// V is never reconstructed per token: by linearity of Eq. 3 the weighted sum is taken in
// spectral space and projected once.
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
  // cycles per tile of the K-score kernel by rank class: a least-squares fit, one coefficient per class, of every CTA's busy
  // time to its tile counts on the benchmark's mix of classes (8 KV heads, CTA pairs; residual 1.3 us rms of 330): a fixed
  // part (rotation factors, the per-slab epilogue and score products) plus a per-panel part, an odd panel count costing a
  // little more than the even one above it saves; classes above 8 run as two passes.  Only the ratios matter.
  constexpr unsigned kCost[TWKV_MAX_CLASSES] = {14300u, 16600u, 18600u, 19500u, 22100u, 23000u, 25400u, 26200u,
                                                38800u, 38700u, 42000u, 42800u, 45600u, 45800u, 49300u, 50700u};
  return kCost[min(max(cls, 1), TWKV_MAX_CLASSES) - 1];
}

// Cut points of one sequence's V tile list into n_splits contiguous ranges of about equal cost (a tile costs its
// panels plus its score rows, counted in 512-byte units): the V pass is bound by the bytes a CTA reads, and tiles of
// classes 1 to 16 dealt out by count alone left the slowest CTA with half as much again as the mean.
// The list is taken in the stride order of vtile_stride(); cut[s] = number of tiles (in that order) whose inclusive cost
// prefix is <= s / n_splits of the total; split s takes positions cut[s] .. cut[s + 1] - 1 of that order.
__device__ void vsplit_plan(const DevView& v, int layer, const int* __restrict__ seq_ids, int qs, int n_splits) {
  __shared__ unsigned long long s_total, s_base;
  __shared__ unsigned s_ws[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seq = seq_ids[qs];
  const int n = (seq >= 0 && seq < v.S) ? v.svc(layer)[seq] : 0;
  const int* list = v.svt(layer) + (size_t)(n > 0 ? seq : 0) * v.TPS;
  const int4* desc = v.desc(layer, 1);
  int* cut = v.vcut + (size_t)qs * (n_splits + 1);
  if (tid == 0) { s_total = 0ull; s_base = 0ull; }
  __syncthreads();
  unsigned mine = 0u;
  const long long stride = vtile_stride(n);
  for (int i = tid; i < n; i += blockDim.x) mine += 32u * (unsigned)desc[list[i]].y + (unsigned)v.Hq;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
  if (lane == 0 && mine) atomicAdd(&s_total, (unsigned long long)mine);
  __syncthreads();
  const unsigned long long W = s_total, ns = (unsigned long long)n_splits;
  if (W == 0ull) {
    for (int s = tid; s <= n_splits; s += blockDim.x) cut[s] = 0;
    return;
  }
  for (int i0 = 0; i0 < n; i0 += blockDim.x) {
    const int i = i0 + tid;
    const unsigned w = i < n ? 32u * (unsigned)desc[list[(int)((i * stride) % n)]].y + (unsigned)v.Hq : 0u;
    unsigned inc = w;                                             // inclusive scan inside the warp, then over the warps
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned a = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += a;
    }
    if (lane == 31) s_ws[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      unsigned wk = s_ws[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned a = __shfl_up_sync(0xffffffffu, wk, o);
        if (lane >= o) wk += a;
      }
      s_ws[lane] = wk;
    }
    __syncthreads();
    if (i < n) {
      const unsigned long long p = s_base + (warp ? s_ws[warp - 1] : 0u) + inc, e = p - w;
      // the splits whose boundary floor(s W / ns) falls in [e, p): they start at this tile
      for (unsigned long long s = (e * ns + W - 1ull) / W; s < ns && s * W / ns < p; ++s) cut[s] = i;
    }
    __syncthreads();
    if (tid == 0) s_base += s_ws[31];
    __syncthreads();
  }
  if (tid == 0) cut[n_splits] = n;
}

// K slot -> V slot of every token of one sequence (the V slots carry the opposite link): the K-score kernel stores a
// token's scores at its V slot, so that the V pass finds a tile's score rows next to each other.  CTA j of the vj CTAs of
// a sequence takes the V tiles j * 8 .. j * 8 + 7, then vj * 8 further on, eight tiles (1024 slots) at a time.
__device__ void vlink_plan(const DevView& v, int layer, const int* __restrict__ seq_ids, int qs, int j, int vj) {
  const int seq = seq_ids[qs];
  if (seq < 0 || seq >= v.S) return;
  const int n = v.svc(layer)[seq];
  const int* list = v.svt(layer) + (size_t)seq * v.TPS;
  const int4* desc = v.desc(layer, 1);
  const int* aux = v.aux(layer, 1);
  const int sub = threadIdx.x >> 7, slot = threadIdx.x & (TILE - 1);
  for (int t = j * 8 + sub; t < n; t += vj * 8) {
    const int vt = list[t];
    if (slot < desc[vt].z) v.kv_link[aux[(size_t)vt * TILE + slot]] = vt * TILE + slot;
  }
}

__global__ void __launch_bounds__(1024) plan_kernel(DevView v, int layer, const int* __restrict__ seq_ids, int n_seq, int n_cta, int pairs,
                                                    int n_splits, int vj) {
  if ((int)blockIdx.x > n_seq) {                                  // the last n_seq * vj CTAs: K slot -> V slot links
    const int idx = (int)blockIdx.x - 1 - n_seq;
    vlink_plan(v, layer, seq_ids, idx / vj, idx % vj, vj);
    return;
  }
  if (blockIdx.x > 0) {                                           // CTAs 1 .. n_seq: the V pass's split plan, one sequence each
    vsplit_plan(v, layer, seq_ids, (int)blockIdx.x - 1, n_splits);
    return;
  }
  __shared__ int s_cls_off[TWKV_MAX_CLASSES + 1], s_kcc[TWKV_MAX_CLASSES];
  __shared__ unsigned s_wsum[32];
  __shared__ unsigned s_base;                                     // entries kept so far
  __shared__ int s_keep[TWKV_MAX_CLASSES];                        // kept tiles per class run (run k = class NC - k)
  __shared__ int s_koff[TWKV_MAX_CLASSES + 1], s_ioff[TWKV_MAX_CLASSES + 1];    // start of run k in the tile list / in the item list
  __shared__ unsigned long long s_coff[TWKV_MAX_CLASSES + 1];     // estimated cost of everything before run k
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int s = tid; s < v.S; s += blockDim.x) v.qslot[s] = -1;
  if (tid < TWKV_MAX_CLASSES) s_keep[tid] = 0;
  // the class counts are read by sixteen threads at once (one thread reading them in a loop pays a memory round trip
  // per class)
  if (tid < v.NC) s_kcc[tid] = v.kcc(layer)[tid];
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int c = v.NC; c >= 1; --c) { s_cls_off[v.NC - c] = run; run += s_kcc[c - 1]; }    // widest class first
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
  // the first rows of U_V^-1 this thread needs do not depend on the sums below: their reads go out first
  const int dp = tid & 63, jg = tid >> 6;
  const int jn = d_kv / MG_JGROUPS, j0 = jg * jn;
  const unsigned* ucol = reinterpret_cast<const unsigned*>(Uinv_v + g * HEAD_DIM) + dp;    // two 16-bit columns per load
  unsigned u[16], un[16];
#pragma unroll
  for (int t = 0; t < 16; ++t) u[t] = __ldg(ucol + (size_t)(j0 + t) * (d_kv / 2));
  // row sums over the splits: warp w takes row w, its lanes read the splits' parts together, lane 0 adds them in split order
  if ((tid >> 5) < REP) {
    const int r = tid >> 5, lane = tid & 31;
    const int qs = qs0 + r / hp, head = head0 + r % hp;
    float l = 0.f;
    for (int s0 = 0; s0 < n_splits; s0 += 32) {
      const float mine = s0 + lane < n_splits ? v.part_l[((size_t)qs * n_splits + s0 + lane) * Hq + head] : 0.f;
      const int n = min(32, n_splits - s0);
      for (int s = 0; s < n; ++s) l += __shfl_sync(0xffffffffu, mine, s);
    }
    if (lane == 0) sInvL[r] = l > 0.f ? 1.f / l : 0.f;
  }
  // split sums in split order: a thread owns four consecutive columns of one row (one 16-byte read per split) and has
  // the reads of eight splits in flight before it adds them (a loop of dependent adds over one read at a time left
  // this kernel waiting for memory latency)
  for (int i0 = tid * 4; i0 < REP * d_kv; i0 += 4 * MG_THREADS) {
    const int hh = i0 / d_kv, j = i0 - hh * d_kv;                     // d_kv is a multiple of 64: the four columns share a row
    const float4* p = reinterpret_cast<const float4*>(
        v.part_acc + (((size_t)(qs0 + hh / hp) * n_splits) * Hq + head0 + hh % hp) * d_kv + j);
    const size_t stride = (size_t)Hq * d_kv / 4;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < n_splits; s0 += 8) {
      float4 t[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) t[u] = s0 + u < n_splits ? __ldg(p + (size_t)(s0 + u) * stride) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (s0 + u < n_splits) { a.x += t[u].x; a.y += t[u].y; a.z += t[u].z; a.w += t[u].w; }
    }
    *reinterpret_cast<float4*>(sAcc + i0) = a;
  }
  __syncthreads();
  for (int i0 = tid * 4; i0 < REP * d_kv; i0 += 4 * MG_THREADS) {       // each thread scales what it wrote
    const float il = sInvL[i0 / d_kv];
    float4 a = *reinterpret_cast<float4*>(sAcc + i0);
    a.x *= il; a.y *= il; a.z *= il; a.w *= il;
    *reinterpret_cast<float4*>(sAcc + i0) = a;
  }
  __syncthreads();
  float o[8][2];
#pragma unroll
  for (int h = 0; h < 8; ++h) { o[h][0] = 0.f; o[h][1] = 0.f; }
  for (int jb = 0; jb < jn; jb += 16) {                // jn is a multiple of 16 (d_kv a multiple of 128)
    if (jb + 16 < jn) {                                // the next sixteen rows are on their way while these are used
#pragma unroll
      for (int t = 0; t < 16; ++t) un[t] = __ldg(ucol + (size_t)(j0 + jb + 16 + t) * (d_kv / 2));
    }
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
#pragma unroll
    for (int t = 0; t < 16; ++t) u[t] = un[t];
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
cudaError_t launch_vacc_tc(const DevView& v, int layer, const CUtensorMap& map_blocks, const CUtensorMap* map_scores, const int* seq_ids,
                           int n_seq, int n_splits, cudaStream_t st);

template <bool BF16>
static cudaError_t launch_decode_t(const DevView& v, int layer, const LayerParams& lp, const void* q, const int* seq_ids,
                                   int n_seq, void* out, int n_splits, int sm_count, const TcMaps* maps, bool pairs, cudaStream_t st) {
  // the K-score kernel's work is cut into one piece per persistent CTA, or per CTA pair
  const int n_pieces = pairs ? kscore_max_pairs(sm_count) : sm_count;
  // CTAs per sequence that invert the V -> K links: enough of them that they finish inside the K work list's time
  const int vj = n_seq >= 256 ? 1 : (256 / n_seq > 64 ? 64 : 256 / n_seq);
  { ProfScope ps(TWKV_K_PLAN, st); plan_kernel<<<1 + n_seq + n_seq * vj, 1024, 0, st>>>(v, layer, seq_ids, n_seq, n_pieces, pairs ? 1 : 0, n_splits, vj); }
  {
    cudaError_t e = launch_kscore_tc(v, layer, maps->blocks, maps->uinvT_k, q, n_pieces, pairs, st);
    if (e != cudaSuccess) return e;
  }
  {
    ProfScope ps(TWKV_K_VACC, st);
    cudaError_t e = launch_vacc_tc(v, layer, maps->blocks, maps->scores, seq_ids, n_seq, n_splits, st);
    if (e != cudaSuccess) return e;
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
