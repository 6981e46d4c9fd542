// Compress step: gate -> rank (Eq. 5, 6, 8), slot allocation, truncate + pack (Eq. 2).
//
// A compress piece (<= TWKV_PIECE_TOKENS = 131072 tokens) runs as: hist (per-chunk key counts) -> alloc (one CTA:
// exclusive scans, capacity check, tile and block allocation in ascending key order) -> pack
// (warp per token: 128-bit loads / stores of the retained prefix, +0 fill to the class width).
// Slot assignment is a function of the token order only (no atomics decide placement), so the
// packed bytes and tables are reproducible.
#include "twkv_dev.h"

namespace twkv {

// ------------------------------------------------------------------------------------------
// Gate: warp per (token, side).  Each lane owns d/32 consecutive logits, so the cumulative sum
// of Eq. 6 is a lane-local running sum plus a warp scan of the lane totals.
//   p = softmax(z) (Eq. 5), c_n = sum_{j<=n} p_j, m_i = c_{d+1-i} (Eq. 6),
//   r = #{i : m_i > tau} = d - #{n : c_n <= tau} (Eq. 8).
// The comparison c_n <= tau is done as S_n <= tau * S_d on the unnormalised sums.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gate_rank_kernel(const float* __restrict__ logits, unsigned short* __restrict__ levels,
                                                        int n_rows, int d, float tau, int* status) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= n_rows) return;
  const int per = d >> 5;                       // 4 .. 32, multiple of 4
  const float* z = logits + (size_t)warp * d + lane * per;
  float v[32];
  float mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    if (i < per) {
      float4 t = *reinterpret_cast<const float4*>(z + i);
      v[i] = t.x; v[i + 1] = t.y; v[i + 2] = t.z; v[i + 3] = t.w;
      mx = fmaxf(mx, fmaxf(fmaxf(t.x, t.y), fmaxf(t.z, t.w)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float run = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    if (i < per) { run += expf(v[i] - mx); v[i] = run; }
  }
  float incl = run;                             // inclusive scan of lane totals
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    float t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  const float total = __shfl_sync(0xffffffffu, incl, 31);
  const float offset = incl - run;
  const float thr = tau * total;
  int below = 0;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    if (i < per) below += (offset + v[i] <= thr) ? 1 : 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(0xffffffffu, below, o);
  int r = d - below;
  if (r < 1) r = 1;                             // only reachable with tau >= 1 or NaN logits
  if (lane == 0) {
    levels[warp] = (unsigned short)r;
    // a row with a NaN or an infinite logit has no softmax: the rank above is a placeholder, the call reports it
    if (status && !(total > 0.f && total < INFINITY)) atomicCAS(status, 0, TWKV_ERR_DEVICE_CHECK);
  }
}

cudaError_t launch_gate_rank(const DevView& v, const float* logits, unsigned short* levels, int n_tok, cudaStream_t st) {
  const int rows = n_tok * 2;
  if (rows == 0) return cudaSuccess;
  const int blocks = (rows + 7) / 8;
  { ProfScope ps(TWKV_K_GATE_RANK, st); gate_rank_kernel<<<blocks, 256, 0, st>>>(logits, levels, rows, v.d_kv, v.tau, v.status); }
  count_launch();
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int key_of(const DevView& v, int side, int seq, int cls) {
  return (side * v.S + seq) * v.NC + (cls - 1);
}

// A compress call is handled piece by piece (TWKV_PIECE_TOKENS tokens), but the kernels below run once for up to
// v.batch pieces: every piece has its own copy of the per-piece scratch, selected here.
__device__ __forceinline__ DevView piece_view(DevView v, int p) {
  v.hist += (size_t)p * v.NK * PIECE_CHUNKS;
  v.key_cnt += (size_t)p * v.NK; v.key_old_fill += (size_t)p * v.NK; v.key_first_id += (size_t)p * v.NK;
  v.key_first_base += (size_t)p * v.NK; v.key_old_last += (size_t)p * v.NK;
  v.pflags += 2 * p;
  return v;
}

// grid: the chunks of all pieces of the launch group (chunk b belongs to piece b / PIECE_CHUNKS)
__global__ void __launch_bounds__(CHUNK_TOKENS) hist_kernel(DevView v0, const int* __restrict__ seq_ids, const int* __restrict__ positions,
                                                            const unsigned short* __restrict__ levels, int n_tok) {
  const DevView v = piece_view(v0, blockIdx.x / PIECE_CHUNKS);
  const int chunk = blockIdx.x % PIECE_CHUNKS;
  const int i = blockIdx.x * CHUNK_TOKENS + threadIdx.x;
  if (i >= n_tok) return;
  const int seq = seq_ids[i];
  const int rk = levels[2 * i], rv = levels[2 * i + 1];
  const int pos = positions[i];
  if (seq < 0 || seq >= v.S || rk < 1 || rk > v.d_kv || rv < 1 || rv > v.d_kv || pos < 0 || pos >= ROPE_LO * ROPE_HI) {
    atomicOr(&v.pflags[1], 1);
    return;
  }
  atomicAdd(&v.hist[(size_t)key_of(v, 0, seq, (rk + PANEL - 1) / PANEL) * PIECE_CHUNKS + chunk], 1);
  atomicAdd(&v.hist[(size_t)key_of(v, 1, seq, (rv + PANEL - 1) / PANEL) * PIECE_CHUNKS + chunk], 1);
}

// Warp per key: the key's per-chunk counts (contiguous, [key][chunk]) become exclusive bases, their sum the key's count.
// grid: one warp per (piece, key); total_chunks counts the chunks of all pieces of the launch group
__global__ void __launch_bounds__(256) scan_kernel(DevView v0, int n_pieces, int total_chunks) {
  const int widx = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (widx >= v0.NK * n_pieces) return;
  const int piece = widx / v0.NK, key = widx - piece * v0.NK;
  const DevView v = piece_view(v0, piece);
  const int n_chunks = min(PIECE_CHUNKS, total_chunks - piece * PIECE_CHUNKS);
  int* h = v.hist + (size_t)key * PIECE_CHUNKS;
  int carry = 0;
  for (int c0 = 0; c0 < n_chunks; c0 += 128) {
    const int c = c0 + lane * 4;
    int4 t = make_int4(0, 0, 0, 0);
    if (c < n_chunks) t = *reinterpret_cast<const int4*>(h + c);          // chunks past n_chunks were cleared
    const int sum = t.x + t.y + t.z + t.w;
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += u;
    }
    const int base = carry + incl - sum;
    if (c < n_chunks) *reinterpret_cast<int4*>(h + c) = make_int4(base, base + t.x, base + t.x + t.y, base + t.x + t.y + t.z);
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) v.key_cnt[key] = carry;
}

__device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// One CTA of 1024 threads, the pieces of the launch group one after the other.  Per piece: checks capacity and, if
// the whole piece fits, creates the new tiles in ascending key order; a piece that does not fit (or holds an invalid
// token) is refused whole and the later pieces carry on from the unchanged tables.
// A call of at most one chunk (the decode-time append) skips the histogram and scan launches: `count_tok` > 0 makes
// this kernel count the call's tokens per key itself (one piece, one chunk, so every per-chunk base is 0).
__global__ void __launch_bounds__(1024) alloc_kernel(DevView v0, int layer, int n_pieces, const int* __restrict__ seq_ids,
                                                     const int* __restrict__ positions, const unsigned short* __restrict__ levels,
                                                     int count_tok) {
  __shared__ int s_scan[3][1024];
  __shared__ int s_fail;
  const int tid = threadIdx.x;
  const int NK = v0.NK;
  int* fill = v0.fill_l(layer);
  int* key_last = v0.key_last_l(layer);
  const int KPT = ceil_div(NK, 1024);
  const int k0 = tid * KPT, k1 = min(NK, k0 + KPT);
  const int half = v0.S * v0.NC;                      // keys per side
  int* ntiles = v0.ntiles(layer);
  int* stok = v0.stok(layer);
  const int warp = tid >> 5, lane = tid & 31;
  if (count_tok > 0) {
    for (int k = k0; k < k1; ++k) v0.key_cnt[k] = 0;
    if (tid < 2) v0.pflags[tid] = 0;
    __syncthreads();
    if (tid < count_tok) {
      const int seq = seq_ids[tid], rk = levels[2 * tid], rv = levels[2 * tid + 1], pos = positions[tid];
      if (seq < 0 || seq >= v0.S || rk < 1 || rk > v0.d_kv || rv < 1 || rv > v0.d_kv || pos < 0 || pos >= ROPE_LO * ROPE_HI) {
        atomicOr(&v0.pflags[1], 1);
      } else {
        const int kk = key_of(v0, 0, seq, (rk + PANEL - 1) / PANEL), kv = key_of(v0, 1, seq, (rv + PANEL - 1) / PANEL);
        atomicAdd(&v0.key_cnt[kk], 1);
        atomicAdd(&v0.key_cnt[kv], 1);
        v0.hist[(size_t)kk * PIECE_CHUNKS] = 0;                // the chunk's base inside the piece
        v0.hist[(size_t)kv * PIECE_CHUNKS] = 0;
      }
    }
    // the barrier at the top of the piece loop publishes the counts
  }
  for (int piece = 0; piece < n_pieces; ++piece) {
    const DevView v = piece_view(v0, piece);
    if (tid == 0) s_fail = 0;
    __syncthreads();                                   // also: the previous piece's table updates are visible
    // (per-key counts and per-chunk bases come from scan_kernel)  new tiles / blocks per key, scanned in key order
    int sum_tk = 0, sum_tv = 0, sum_b = 0;
    for (int k = k0; k < k1; ++k) {
      const int cnt = v.key_cnt[k], old = fill[k];
      v.key_old_fill[k] = old;
      const int nnew = ceil_div(old + cnt, TILE) - ceil_div(old, TILE);
      if (k < half) sum_tk += nnew; else sum_tv += nnew;
      sum_b += nnew * (k % v.NC + 1);
    }
    s_scan[0][tid] = sum_tk; s_scan[1][tid] = sum_tv; s_scan[2][tid] = sum_b;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {                 // inclusive Hillis-Steele scan
      int a = 0, b = 0, c = 0;
      if (tid >= o) { a = s_scan[0][tid - o]; b = s_scan[1][tid - o]; c = s_scan[2][tid - o]; }
      __syncthreads();
      s_scan[0][tid] += a; s_scan[1][tid] += b; s_scan[2][tid] += c;
      __syncthreads();
    }
    const int tot_tk = s_scan[0][1023], tot_tv = s_scan[1][1023], tot_b = s_scan[2][1023];
    const int next_block = v.status[1];
    const int ntk = ntiles[0], ntv = ntiles[1];
    // capacity: tokens per sequence
    for (int s = tid; s < v.S; s += 1024) {
      int add = 0;
      for (int c = 0; c < v.NC; ++c) add += v.key_cnt[s * v.NC + c];
      if (stok[s] + add > v.tmax) atomicOr(&s_fail, 1);
    }
    if (tid == 0) {
      if (next_block + tot_b > v.n_blocks || ntk + tot_tk > v.NT || ntv + tot_tv > v.NT) atomicOr(&s_fail, 1);
      if (v.pflags[1]) atomicOr(&s_fail, 2);
    }
    __syncthreads();
    if (s_fail) {
      if (tid == 0) {
        v.pflags[0] = 0;
        set_status(v, (s_fail & 2) ? TWKV_ERR_INVALID_ARG : TWKV_ERR_CAPACITY);
      }
      __syncthreads();                                 // s_fail is reset at the top of the next round
      continue;
    }
    // commit
    int off_tk = s_scan[0][tid] - sum_tk, off_tv = s_scan[1][tid] - sum_tv, off_b = s_scan[2][tid] - sum_b;
    for (int k = k0; k < k1; ++k) {
      const int cnt = v.key_cnt[k], old = v.key_old_fill[k];
      const int side = k >= half ? 1 : 0;
      const int cls = k % v.NC + 1;
      const int seq = (k / v.NC) % v.S;
      const int old_tiles = ceil_div(old, TILE);
      const int nnew = ceil_div(old + cnt, TILE) - old_tiles;
      const int first_id = (side ? ntv + off_tv : ntk + off_tk);
      const int first_base = next_block + off_b;
      v.key_first_id[k] = first_id;
      v.key_first_base[k] = first_base;
      v.key_old_last[k] = key_last[k];
      if (cnt > 0) {
        const int nf = old + cnt;
        int4* desc = v.desc(layer, side);
        if (old % TILE != 0) desc[key_last[k]].z = min(TILE, nf - (old_tiles - 1) * TILE);
        for (int j = 0; j < nnew; ++j)
          desc[first_id + j] = make_int4(seq, cls, min(TILE, nf - (old_tiles + j) * TILE), first_base + j * cls);
        if (nnew > 0) key_last[k] = first_id + nnew - 1;
        fill[k] = nf;
      }
      if (side) off_tv += nnew; else off_tk += nnew;
      off_b += nnew * cls;
    }
    __syncthreads();
    // tile lists: K per class (ascending sequence), V per sequence (ascending class); one warp per list, one lane per
    // key of the list: the lanes read their keys' tables together, a warp scan places their runs of tile ids
    if (warp < v.NC) {
      int* cnt = v.kcc(layer);
      int* list = v.kct(layer) + (size_t)warp * v.NT;
      int run = cnt[warp];
      for (int s0 = 0; s0 < v.S; s0 += 32) {
        const int s = s0 + lane;
        int nnew = 0, first = 0;
        if (s < v.S) {
          const int k = s * v.NC + warp;
          const int c = v.key_cnt[k], old = v.key_old_fill[k];
          nnew = ceil_div(old + c, TILE) - ceil_div(old, TILE);
          first = v.key_first_id[k];
        }
        int incl = nnew;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int u = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += u;
        }
        int* dst = list + run + incl - nnew;
        for (int j = 0; j < nnew; ++j) dst[j] = first + j;
        run += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) cnt[warp] = run;
    }
    for (int s = warp; s < v.S; s += 32) {
      int* list = v.svt(layer) + (size_t)s * v.TPS;
      const int run0 = v.svc(layer)[s];
      int nnew = 0, first = 0, add = 0;
      if (lane < v.NC) {
        const int k = half + s * v.NC + lane;
        const int cn = v.key_cnt[k], old = v.key_old_fill[k];
        nnew = ceil_div(old + cn, TILE) - ceil_div(old, TILE);
        first = v.key_first_id[k];
        add = v.key_cnt[s * v.NC + lane];
      }
      int incl = nnew;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += u;
        add += __shfl_xor_sync(0xffffffffu, add, o);              // butterfly: every lane ends with the total
      }
      int* dst = list + run0 + incl - nnew;
      for (int j = 0; j < nnew; ++j) dst[j] = first + j;
      if (lane == 31) {
        v.svc(layer)[s] = run0 + incl;
        stok[s] += add;
      }
    }
    if (tid == 0) {
      v.status[1] = next_block + tot_b;
      ntiles[0] = ntk + tot_tk;
      ntiles[1] = ntv + tot_tv;
      v.pflags[0] = 1;
    }
    __syncthreads();
  }
}

struct Place { int base, slot_cls_r; };   // slot | cls << 8 | r << 16

// grid: the chunks of all pieces of the launch group (chunk b belongs to piece b / PIECE_CHUNKS), then one CTA per
// (piece, key) for the tile tails
__global__ void __launch_bounds__(CHUNK_TOKENS, 7) pack_kernel(DevView v0, int layer, const void* __restrict__ K, const void* __restrict__ V,
                                                            const int* __restrict__ seq_ids, const int* __restrict__ positions,
                                                            const unsigned short* __restrict__ levels, int n_tok) {
  const int n_chunks = (n_tok + CHUNK_TOKENS - 1) / CHUNK_TOKENS;
  const bool tail_cta = (int)blockIdx.x >= n_chunks;
  const int piece = tail_cta ? (blockIdx.x - n_chunks) / v0.NK : blockIdx.x / PIECE_CHUNKS;
  const DevView v = piece_view(v0, piece);
  if (v.pflags[0] == 0) return;                           // the piece was refused
  const int chunk = blockIdx.x % PIECE_CHUNKS;            // of a token CTA, inside its piece
  if (tail_cta) {
    // one CTA per (piece, key): if the key's last token of the piece sits in a tile created by the piece and the
    // tile is not full, zero the slots behind it (decode reads whole tiles).
    const int k = (blockIdx.x - n_chunks) % v.NK;
    const int cnt = v.key_cnt[k];
    if (cnt == 0) return;
    const int old = v.key_old_fill[k], cls = k % v.NC + 1;
    const int g = old + cnt - 1, ord = g / TILE, slot = g % TILE, old_tiles = (old + TILE - 1) / TILE;
    if (ord < old_tiles) return;
    // later pieces of this launch group keep filling the same tile (their CTAs run beside this one): leave them
    // their slots and zero from behind the key's last token of the whole group
    int later = 0;
    const int n_pieces = (n_chunks + PIECE_CHUNKS - 1) / PIECE_CHUNKS;
    for (int q = piece + 1; q < n_pieces; ++q) {
      const DevView w = piece_view(v0, q);
      if (w.pflags[0]) later += w.key_cnt[k];
    }
    const int first_zero = slot + 1 + later;
    if (first_zero >= TILE) return;
    const int base = v.key_first_base[k] + (ord - old_tiles) * cls;
    const int n16 = (TILE - first_zero) * 8;               // 16-byte chunks behind the last token, per panel
    for (int panel = 0; panel < cls; ++panel) {
      uint4* dst = reinterpret_cast<uint4*>(v.blocks + (size_t)(base + panel) * BLOCK_BYTES + first_zero * (PANEL * 2));
      for (int i = threadIdx.x; i < n16; i += CHUNK_TOKENS) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    return;
  }
  __shared__ int s_key[2][CHUNK_TOKENS];
  __shared__ Place s_place[2][CHUNK_TOKENS];
  __shared__ unsigned long long s_sum[2];
  const int tid = threadIdx.x;
  const int i = blockIdx.x * CHUNK_TOKENS + tid;
  const bool valid = i < n_tok;
  int seq = 0, r[2] = {1, 1};
  if (valid) { seq = seq_ids[i]; r[0] = levels[2 * i]; r[1] = levels[2 * i + 1]; }
  int key[2];
#pragma unroll
  for (int side = 0; side < 2; ++side) {
    key[side] = valid ? key_of(v, side, seq, (r[side] + PANEL - 1) / PANEL) : -1 - side;
    s_key[side][tid] = key[side];
  }
  if (tid < 2) s_sum[tid] = 0ull;
  __syncthreads();
  int before[2] = {0, 0};
  for (int j = 0; j < tid; ++j) {
    before[0] += (s_key[0][j] == key[0]) ? 1 : 0;
    before[1] += (s_key[1][j] == key[1]) ? 1 : 0;
  }
  if (valid) {
    int kslot = 0;
#pragma unroll
    for (int side = 0; side < 2; ++side) {
      const int k = key[side];
      const int cls = k % v.NC + 1;
      const int old = v.key_old_fill[k];
      const int g = old + v.hist[(size_t)k * PIECE_CHUNKS + chunk] + before[side];
      const int ord = g / TILE, slot = g % TILE;
      const int old_tiles = (old + TILE - 1) / TILE;
      int tile, base;
      const bool is_new = ord >= old_tiles;
      if (is_new) {
        tile = v.key_first_id[k] + (ord - old_tiles);
        base = v.key_first_base[k] + (ord - old_tiles) * cls;
      } else {
        tile = v.key_old_last[k];
        base = v.desc(layer, side)[tile].w;
      }
      s_place[side][tid].base = base;
      s_place[side][tid].slot_cls_r = slot | (cls << 8) | (r[side] << 16);
      v.rank(layer, side)[(size_t)tile * TILE + slot] = (unsigned short)r[side];
      if (side == 0) {
        v.aux(layer, 0)[(size_t)tile * TILE + slot] = positions[i];
        kslot = tile * TILE + slot;
      } else {
        v.aux(layer, 1)[(size_t)tile * TILE + slot] = kslot;
      }
    }
  }
  {
    unsigned rk = valid ? (unsigned)r[0] : 0u, rv = valid ? (unsigned)r[1] : 0u;          // <= 32 * 1024 per warp
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { rk += __shfl_xor_sync(0xffffffffu, rk, o); rv += __shfl_xor_sync(0xffffffffu, rv, o); }
    if ((tid & 31) == 0) { atomicAdd(&s_sum[0], (unsigned long long)rk); atomicAdd(&s_sum[1], (unsigned long long)rv); }
  }
  __syncthreads();
  if (tid < 2 && s_sum[tid]) atomicAdd(&v.rank_sums[layer * 2 + tid], s_sum[tid]);
  // Move the rows.  The CTA's 256 (token, side) rows are a flat list of 16-byte chunks (8 elements; a row of class c
  // has 8 c of them, those past the rank are zero fill); thread i takes chunks i, i + 128, ... so every lane has
  // work whatever the rows' widths, and loads PACK_UNROLL chunks before it stores any.
  // Every row is a whole number of 8-chunk groups (one 128-byte panel row each); s_oct maps a group to its row and to
  // the panel inside the row, so finding a chunk's row is one shared-memory read.
  __shared__ unsigned short s_oct[2 * CHUNK_TOKENS * TWKV_MAX_CLASSES];      // (row << 4) | panel
  __shared__ int s_total;
  __shared__ int s_wtot[CHUNK_TOKENS / 32];
  {
    const int c0 = valid ? ((s_place[0][tid].slot_cls_r >> 8) & 0xff) * 8 : 0;
    const int c1 = valid ? ((s_place[1][tid].slot_cls_r >> 8) & 0xff) * 8 : 0;
    int inc = c0 + c1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, o);
      if ((tid & 31) >= o) inc += n;
    }
    if ((tid & 31) == 31) s_wtot[tid >> 5] = inc;
    __syncthreads();
    int off = 0;
    for (int w = 0; w < (tid >> 5); ++w) off += s_wtot[w];
    const int excl = off + inc - (c0 + c1);
    for (int pnl = 0; pnl < (c0 >> 3); ++pnl) s_oct[(excl >> 3) + pnl] = (unsigned short)(((2 * tid) << 4) | pnl);
    for (int pnl = 0; pnl < (c1 >> 3); ++pnl) s_oct[((excl + c0) >> 3) + pnl] = (unsigned short)(((2 * tid + 1) << 4) | pnl);
    if (tid == CHUNK_TOKENS - 1) s_total = excl + c0 + c1;
  }
  __syncthreads();
  const int total = s_total;
  const size_t row_bytes = (size_t)v.d_kv * 2;
  constexpr int PACK_UNROLL = 8;
  for (int cb = tid; cb < total; cb += CHUNK_TOKENS * PACK_UNROLL) {
    uint4 val[PACK_UNROLL];
    unsigned char* dst[PACK_UNROLL];
    int keep[PACK_UNROLL];
#pragma unroll
    for (int u = 0; u < PACK_UNROLL; ++u) {
      const int c = cb + u * CHUNK_TOKENS;
      val[u] = make_uint4(0u, 0u, 0u, 0u);
      dst[u] = nullptr;
      keep[u] = 8;
      if (c < total) {
        const int info = s_oct[c >> 3];
        const int t = info >> 5, side = (info >> 4) & 1, j = (info & 15) * 8 + (c & 7);
        const Place p = s_place[side][t];
        const int slot = p.slot_cls_r & 0xff, rr = p.slot_cls_r >> 16;
        keep[u] = rr - j * 8;
        if (keep[u] > 0)
          val[u] = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(side ? V : K) +
                                                        (size_t)(blockIdx.x * CHUNK_TOKENS + t) * row_bytes) + j);
        dst[u] = v.blocks + (size_t)(p.base + (j >> 3)) * BLOCK_BYTES + slot * (PANEL * 2) + (j & 7) * 16;
      }
    }
#pragma unroll
    for (int u = 0; u < PACK_UNROLL; ++u) {
      if (!dst[u]) continue;
      uint4 o = val[u];
      if (keep[u] < 8) {                                         // elements kept in this chunk
        unsigned* w = reinterpret_cast<unsigned*>(&o);
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          const int left = keep[u] - 2 * p;
          if (left <= 0) w[p] = 0u;
          else if (left == 1) w[p] &= 0x0000ffffu;
        }
      }
      *reinterpret_cast<uint4*>(dst[u]) = o;
    }
  }
}

// The pieces of up to v.batch * TWKV_PIECE_TOKENS tokens: one launch each of the histogram, the per-key scan, the
// allocator (which takes the pieces in order) and the packer.
cudaError_t launch_compress_pieces(const DevView& v, int layer, const void* K, const void* V, const int* seq_ids,
                                   const int* positions, int n_tok, const unsigned short* levels, cudaStream_t st) {
  if (n_tok <= 0) return cudaSuccess;
  const int n_chunks = (n_tok + CHUNK_TOKENS - 1) / CHUNK_TOKENS;
  const int n_pieces = (n_chunks + PIECE_CHUNKS - 1) / PIECE_CHUNKS;
  // scan_kernel reads the counts four at a time; a launch group of several pieces clears its tables whole
  if (n_chunks == 1) {
    // decode-time append: the allocator counts the tokens itself, two launches in all
    { ProfScope ps(TWKV_K_ALLOC, st); alloc_kernel<<<1, 1024, 0, st>>>(v, layer, 1, seq_ids, positions, levels, n_tok); }
    { ProfScope ps(TWKV_K_PACK, st); pack_kernel<<<1 + v.NK, CHUNK_TOKENS, 0, st>>>(v, layer, K, V, seq_ids, positions, levels, n_tok); }
    count_launch(2);
    return cudaGetLastError();
  }
  const int n_cols = n_pieces > 1 ? PIECE_CHUNKS : (n_chunks + 3) & ~3;
  cudaError_t e = cudaMemset2DAsync(v.hist, (size_t)PIECE_CHUNKS * sizeof(int), 0, (size_t)n_cols * sizeof(int), (size_t)v.NK * n_pieces, st);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(v.pflags, 0, (size_t)v.batch * 2 * sizeof(int), st);
  if (e != cudaSuccess) return e;
  { ProfScope ps(TWKV_K_HIST, st); hist_kernel<<<n_chunks, CHUNK_TOKENS, 0, st>>>(v, seq_ids, positions, levels, n_tok); }
  {
    ProfScope ps(TWKV_K_ALLOC, st);
    scan_kernel<<<(v.NK * n_pieces + 7) / 8, 256, 0, st>>>(v, n_pieces, n_chunks);
    alloc_kernel<<<1, 1024, 0, st>>>(v, layer, n_pieces, nullptr, nullptr, nullptr, 0);
  }
  { ProfScope ps(TWKV_K_PACK, st); pack_kernel<<<n_chunks + v.NK * n_pieces, CHUNK_TOKENS, 0, st>>>(v, layer, K, V, seq_ids, positions, levels, n_tok); }
  count_launch(4);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Two-level RoPE tables, built once per cache in fp64: angle(pos, i) = pos * base^(-2i/128), pos = hi * 16 + lo.
// cos/sin of the sum come from the angle-addition formulas at use (one complex product per frequency); the 16 `lo`
// rows fit in shared memory, the 8 KB-apart `hi` rows a tile touches stay in L2 (1 MiB per 32768 positions).
// Entries are stored per pair of frequencies as (cos, cos, sin, sin), the packed form the K-score kernel multiplies.
// ------------------------------------------------------------------------------------------
__global__ void rope_tables_kernel(float4* lo, float4* hi, double base) {
  const int t = threadIdx.x;                                   // frequency pair (2 t, 2 t + 1)
  const int row = blockIdx.x;
  const double th0 = pow(base, -2.0 * (double)(2 * t) / (double)HEAD_DIM), th1 = pow(base, -2.0 * (double)(2 * t + 1) / (double)HEAD_DIM);
  double s0, c0, s1, c1;
  if (row < ROPE_LO) {
    sincos((double)row * th0, &s0, &c0);
    sincos((double)row * th1, &s1, &c1);
    lo[row * 32 + t] = make_float4((float)c0, (float)c1, (float)s0, (float)s1);
  }
  sincos((double)row * (double)ROPE_LO * th0, &s0, &c0);
  sincos((double)row * (double)ROPE_LO * th1, &s1, &c1);
  hi[(size_t)row * 32 + t] = make_float4((float)c0, (float)c1, (float)s0, (float)s1);
}

cudaError_t launch_rope_tables(const DevView& v, float rope_base, cudaStream_t st) {
  rope_tables_kernel<<<ROPE_HI, 32, 0, st>>>(v.rope_lo, v.rope_hi, (double)rope_base);
  count_launch();
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Statistics: tokens per class from the fill table, rank sums, blocks in use.
// out[0] tokens, [1] bytes_stored, [2] sum r_K, [3] sum r_V, [4] blocks used, [5 ..] tokens_per_class[2][16]
// ------------------------------------------------------------------------------------------
__global__ void stats_kernel(DevView v, int layer, unsigned long long* out) {
  const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? v.L : layer + 1;
  for (int i = threadIdx.x; i < 5 + 2 * TWKV_MAX_CLASSES; i += blockDim.x) out[i] = 0ull;
  __syncthreads();
  const int half = v.S * v.NC;
  for (int l = l0; l < l1; ++l) {
    const int* fill = v.fill_l(l);
    for (int k = threadIdx.x; k < v.NK; k += blockDim.x) {
      const unsigned long long f = (unsigned long long)fill[k];
      if (!f) continue;
      const int side = k >= half, cls = k % v.NC + 1;
      atomicAdd(&out[5 + side * TWKV_MAX_CLASSES + cls - 1], f);
      atomicAdd(&out[1], f * (unsigned long long)(cls * PANEL * 2));
      if (!side) atomicAdd(&out[0], f);
    }
    if (threadIdx.x == 0) {
      atomicAdd(&out[2], v.rank_sums[l * 2]);
      atomicAdd(&out[3], v.rank_sums[l * 2 + 1]);
    }
  }
  if (threadIdx.x == 0) out[4] = (unsigned long long)v.status[1];
}

cudaError_t launch_stats(const DevView& v, int layer, unsigned long long* out_dev, cudaStream_t st) {
  stats_kernel<<<1, 256, 0, st>>>(v, layer, out_dev);
  count_launch();
  return cudaGetLastError();
}

}  // namespace twkv
