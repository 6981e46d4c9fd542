// Global token eviction (the paper's combination with token eviction, Sec. 5.2 "Implementation Details": the spectral
// decomposition is joint across heads, so a token is kept or dropped for all heads at once) and compaction of the
// survivors inside the cache.
//
//   twkv_evict(cache, layer, seq, keep_positions, n_keep): of the tokens cached for `seq` in `layer`, exactly those
//   whose position is listed survive, on the K side and on the V side.
// Container rule.  For every (side, class) of the sequence the survivors move to the front of the tiles that key
// already owns, in their stored order; the vacated rows of the last tile that stays in use are zeroed; tiles left
// without a token are taken off the tile lists (their blocks stay unused until the cache is reset).  V slots are
// relinked to the new slots of their tokens' K rows.  Later appends continue behind the survivors.
//
// Four launches: (1) bitmap of the kept positions; (2) per key, the destination of every slot (nothing moves yet: the
// V side finds a token's position through its K row); (3) per key, the moves (a tile's rows are all read before any is
// written, destinations never lie behind sources); (4) the tile lists without the emptied tiles.
#include "twkv_dev.h"

namespace twkv {

constexpr int EV_THREADS = 1024;

// exclusive scan of one value per thread over the CTA; returns the thread's offset, *total = sum (valid for all threads)
__device__ __forceinline__ int block_scan_excl(int x, int* s_warp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += u;
  }
  __syncthreads();                                         // s_warp may still be read from the previous call
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += u;
    }
    s_warp[lane] = w;
  }
  __syncthreads();
  *total = s_warp[31];
  return (warp ? s_warp[warp - 1] : 0) + incl - x;
}

// The tiles of key (side, seq, cls) in creation order -> s_tiles; returns their number.  K tiles are listed per class
// (all sequences), V tiles per sequence (all classes); both lists are in creation order.
__device__ int collect_key_tiles(const DevView& v, int layer, int side, int seq, int cls, int* s_tiles, int* s_warp) {
  const int4* desc = v.desc(layer, side);
  const int* list = side ? v.svt(layer) + (size_t)seq * v.TPS : v.kct(layer) + (size_t)(cls - 1) * v.NT;
  const int n = side ? v.svc(layer)[seq] : v.kcc(layer)[cls - 1];
  int base = 0;
  for (int i0 = 0; i0 < n; i0 += EV_THREADS) {
    const int i = i0 + threadIdx.x;
    int t = -1, mine = 0;
    if (i < n) {
      t = list[i];
      const int4 d = desc[t];
      mine = (d.x == seq && d.y == cls) ? 1 : 0;
    }
    int total;
    const int off = block_scan_excl(mine, s_warp, &total);
    if (mine) s_tiles[base + off] = t;
    base += total;
  }
  __syncthreads();
  return base;
}

__global__ void __launch_bounds__(EV_THREADS) evict_bitmap_kernel(DevView v, int layer, int seq, const int* __restrict__ keep, int n_keep) {
  unsigned* bm = v.evict_bitmap;
  for (int i = threadIdx.x; i < (ROPE_LO * ROPE_HI) / 32; i += EV_THREADS) bm[i] = 0u;
  __syncthreads();
  for (int i = threadIdx.x; i < n_keep; i += EV_THREADS) {
    const int p = keep[i];
    if (p >= 0 && p < ROPE_LO * ROPE_HI) atomicOr(&bm[p >> 5], 1u << (p & 31));
  }
  if (threadIdx.x == 0) v.stok(layer)[seq] = 0;            // the K-side keys add their survivors back
}

// grid (NC, 2): one CTA per key of the sequence.  evict_map[side][tile * 128 + slot] = new global slot, or -1.
__global__ void __launch_bounds__(EV_THREADS) evict_plan_kernel(DevView v, int layer, int seq) {
  extern __shared__ int s_tiles[];
  __shared__ int s_warp[32];
  const int cls = blockIdx.x + 1, side = blockIdx.y, tid = threadIdx.x;
  const int nk = collect_key_tiles(v, layer, side, seq, cls, s_tiles, s_warp);
  const int4* desc = v.desc(layer, side);
  const int* aux = v.aux(layer, side);
  const int* kaux = v.aux(layer, 0);
  const unsigned short* rank = v.rank(layer, side);
  int* map = v.evict_map + (size_t)side * v.NT * TILE;
  int base = 0;
  unsigned long long dropped = 0ull;
  for (int j0 = 0; j0 < nk; j0 += EV_THREADS / TILE) {
    const int j = j0 + tid / TILE, slot = tid % TILE;
    int keep = 0, t = -1;
    if (j < nk) {
      t = s_tiles[j];
      if (slot < desc[t].z) {
        const int a = aux[(size_t)t * TILE + slot];
        const int pos = side ? kaux[a] : a;                // a V slot links to its token's K slot, which holds the position
        keep = (v.evict_bitmap[pos >> 5] >> (pos & 31)) & 1u;
        if (!keep) dropped += rank[(size_t)t * TILE + slot];
      }
    }
    int total;
    const int off = block_scan_excl(keep, s_warp, &total);
    if (t >= 0) {
      const int g = base + off;
      map[(size_t)t * TILE + slot] = keep ? s_tiles[g / TILE] * TILE + g % TILE : -1;
    }
    base += total;
  }
  // dropped ranks leave the layer's rank sums (Eq. 4 statistics)
  for (int o = 16; o > 0; o >>= 1) dropped += __shfl_xor_sync(0xffffffffu, dropped, o);
  if ((tid & 31) == 0 && dropped) atomicAdd(&v.rank_sums[layer * 2 + side], 0ull - dropped);
  if (tid == 0) {
    const int key = (side * v.S + seq) * v.NC + (cls - 1);
    v.evict_fill[side * v.NC + cls - 1] = base;             // the move kernel commits it
    v.key_last_l(layer)[key] = base > 0 ? s_tiles[(base - 1) / TILE] : -1;
    if (side == 0 && base) atomicAdd(&v.stok(layer)[seq], base);
  }
}

// grid (NC, 2): the moves of one key.  Source tiles are taken in order, one tile per round: every row (and its
// position / link and rank) is read into registers, the CTA synchronises, then the survivors are written.
__global__ void __launch_bounds__(EV_THREADS) evict_move_kernel(DevView v, int layer, int seq) {
  extern __shared__ int s_tiles[];
  __shared__ int s_warp[32];
  const int cls = blockIdx.x + 1, side = blockIdx.y, tid = threadIdx.x;
  const int nk = collect_key_tiles(v, layer, side, seq, cls, s_tiles, s_warp);
  int4* desc = v.desc(layer, side);
  int* aux = v.aux(layer, side);
  unsigned short* rank = v.rank(layer, side);
  const int* map = v.evict_map + (size_t)side * v.NT * TILE;
  const int* kmap = v.evict_map;
  const int new_fill = v.evict_fill[side * v.NC + cls - 1];
  const int per_row = cls * 8;                              // 16-byte pieces per stored row
  for (int j = 0; j < nk; ++j) {
    const int t = s_tiles[j];
    const int sbase = desc[t].w;
    // this thread's 16 bytes of every panel: row tid / 8, piece tid % 8; panels are separate blocks, so each is read,
    // synchronised and written on its own
    const int slot = tid >> 3;
    const int to = map[(size_t)t * TILE + slot];
    const bool moves = to >= 0 && to != t * TILE + slot;
    const size_t src_off = (size_t)sbase * BLOCK_BYTES + slot * 128 + (tid & 7) * 16;
    const size_t dst_off = moves ? (size_t)desc[to / TILE].w * BLOCK_BYTES + (to % TILE) * 128 + (tid & 7) * 16 : 0;
    int a = 0, to_slot = -1;
    unsigned short r = 0;
    if (tid < TILE) {
      to_slot = map[(size_t)t * TILE + tid];
      if (to_slot >= 0) {
        a = aux[(size_t)t * TILE + tid];
        if (side) a = kmap[a];                               // the token's K row has moved too
        r = rank[(size_t)t * TILE + tid];
      }
    }
    for (int p = 0; p < cls; ++p) {
      uint4 piece = make_uint4(0u, 0u, 0u, 0u);
      if (moves) piece = *reinterpret_cast<const uint4*>(v.blocks + src_off + (size_t)p * BLOCK_BYTES);
      __syncthreads();
      if (moves) *reinterpret_cast<uint4*>(v.blocks + dst_off + (size_t)p * BLOCK_BYTES) = piece;
    }
    if (to_slot >= 0) { aux[to_slot] = a; rank[to_slot] = r; }       // (read before the first barrier of the panel loop)
    __syncthreads();
  }
  // rows behind the last survivor in the last tile still in use are zero, as after an append
  const int kept = (new_fill + TILE - 1) / TILE;
  if (kept > 0 && new_fill % TILE) {
    const int t = s_tiles[kept - 1], first = new_fill % TILE, base = desc[t].w;
    for (int q = tid; q < (TILE - first) * per_row; q += EV_THREADS) {
      const int slot = first + q / per_row, within = q % per_row;
      *reinterpret_cast<uint4*>(v.blocks + (size_t)(base + (within >> 3)) * BLOCK_BYTES + slot * 128 + (within & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  __syncthreads();
  for (int j = tid; j < nk; j += EV_THREADS) desc[s_tiles[j]].z = j < kept ? min(TILE, new_fill - j * TILE) : 0;
  if (tid == 0) v.fill_l(layer)[(side * v.S + seq) * v.NC + (cls - 1)] = new_fill;
}

// grid NC + 1: the K tile list of every class, and the sequence's V tile list, without the emptied tiles of `seq`
__global__ void __launch_bounds__(EV_THREADS) evict_lists_kernel(DevView v, int layer, int seq) {
  __shared__ int s_warp[32];
  const bool vlist = (int)blockIdx.x == v.NC;
  const int side = vlist ? 1 : 0;
  const int4* desc = v.desc(layer, side);
  int* list = vlist ? v.svt(layer) + (size_t)seq * v.TPS : v.kct(layer) + (size_t)blockIdx.x * v.NT;
  int* count = vlist ? v.svc(layer) + seq : v.kcc(layer) + blockIdx.x;
  const int n = *count;
  int base = 0;
  for (int i0 = 0; i0 < n; i0 += EV_THREADS) {
    const int i = i0 + threadIdx.x;
    int t = -1, stay = 0;
    if (i < n) {
      t = list[i];
      const int4 d = desc[t];
      stay = (d.x == seq && d.z == 0) ? 0 : 1;
    }
    int total;
    const int off = block_scan_excl(stay, s_warp, &total);   // (its barriers also separate this round's reads from the writes)
    if (stay) list[base + off] = t;
    base += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) *count = base;
}

cudaError_t launch_evict(const DevView& v, int layer, int seq, const int* keep_positions, int n_keep, cudaStream_t st) {
  const size_t smem = (size_t)v.TPS * sizeof(int);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(evict_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(evict_move_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  ProfScope ps(TWKV_K_OTHER, st);
  evict_bitmap_kernel<<<1, EV_THREADS, 0, st>>>(v, layer, seq, keep_positions, n_keep);
  evict_plan_kernel<<<dim3(v.NC, 2), EV_THREADS, smem, st>>>(v, layer, seq);
  evict_move_kernel<<<dim3(v.NC, 2), EV_THREADS, smem, st>>>(v, layer, seq);
  evict_lists_kernel<<<v.NC + 1, EV_THREADS, 0, st>>>(v, layer, seq);
  count_launch(4);
  return cudaGetLastError();
}

}  // namespace twkv
