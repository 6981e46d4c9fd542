// Internal definitions shared by the libtwkv translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "twkv.h"

namespace twkv {

constexpr int TILE = TWKV_TILE_TOKENS;      // tokens per tile (the MMA M)
constexpr int PANEL = TWKV_PANEL_ELEMS;     // elements per panel row
constexpr int BLOCK_BYTES = TWKV_BLOCK_BYTES;
constexpr int HEAD_DIM = 128;
constexpr int CHUNK_TOKENS = 128;           // tokens per compress CTA
constexpr int PIECE_CHUNKS = TWKV_PIECE_TOKENS / CHUNK_TOKENS;
constexpr int ROPE_LO = 16;                 // pos = hi * 16 + lo
constexpr int ROPE_HI = 32768;              // positions up to 16 * 32768 - 1
constexpr int MAX_PARTIALS_EXTRA = 320;     // V-side partial slots beyond max_seqs
constexpr int MAX_PLAN_CTAS = 1024;         // upper bound on the K-score kernel's grid
constexpr unsigned long long TWKV_GUARD_WORD = 0x7477b2006b765f67ull;   // written behind every region of the pool

// Device view of a cache: plain pointers into the caller's pool.  Passed to kernels by value.
struct DevView {
  int L, Hq, Hkv, rep, d_kv, NC, S, tmax, NT, TPS, n_blocks, dtype, out_dtype, NK, max_partials;
  float tau, sm_scale;
  int debug;                 // TWKV_DEBUG=1 at cache creation: extra device-side checks (rotated keys inside the f16 range)
  int* status;               // [8]: [0] sticky status, [1] next free block, [2] rows listed for the gate fix-up, [3] its finished CTAs
  int* pflags;               // [batch][2]: piece accepted, piece holds an invalid token (scratch of one compress call)
  int batch;                 // pieces of a compress call whose bookkeeping is launched together
  // RoPE tables, one float4 per pair of frequencies (2t, 2t + 1): (cos_2t, cos_2t+1, sin_2t, sin_2t+1)
  float4* rope_lo;           // [ROPE_LO][32]  angles lo * theta_i
  float4* rope_hi;           // [ROPE_HI][32]  angles hi * 16 * theta_i
  unsigned char* blocks;     // n_blocks x 16 KiB
  // per-layer tables (index with the helpers below)
  int* n_tiles;              // [L][2]
  int4* tile_desc;           // [L][2][NT]  (seq, class, n_valid, base block)
  int* tile_aux;             // [L][2][NT][128]
  unsigned short* tile_rank; // [L][2][NT][128]
  int* fill;                 // [L][NK]
  int* key_last;             // [L][NK]  id of the key's newest tile, -1 if none
  int* kclass_count;         // [L][NC]
  int* kclass_tiles;         // [L][NC][NT]
  int* seq_vcount;           // [L][S]
  int* seq_vtiles;           // [L][S][TPS]
  int* seq_tokens;           // [L][S]
  unsigned long long* rank_sums;  // [L][2]  sum of r_K, r_V
  // scratch shared by all layers
  // per-piece scratch of a compress call, [batch] copies each (piece_view() selects one)
  int* hist;                 // [NK][PIECE_CHUNKS]   per-chunk key counts -> exclusive bases
  int* key_cnt;              // [NK]  tokens of the key in the piece
  int* key_old_fill;         // [NK]  tokens of the key before the piece
  int* key_first_id;         // [NK]  id of the key's first new tile
  int* key_first_base;       // [NK]  base block of the key's first new tile
  int* key_old_last;         // [NK]  the key's newest tile before the piece
  float* scores;             // [NT*128][Hq]  row = V slot of the token (the V pass reads a tile's rows together)
  unsigned* seqmax;          // [S][Hq]  order-preserving encoding of the running max
  int* qslot;                // [S]   sequence id -> query index of the current decode call, -1
  // chunked prefill (null for a decode call): per query slot, the row of q / out it stands for and the last position it
  // may attend to
  const int* qmap;
  const int* qpos;
  // scratch of twkv_evict
  unsigned* evict_bitmap;    // one bit per position: the positions that stay
  int* evict_map;            // [2][NT * 128]  new global slot of every K / V slot of the sequence, -1 = dropped
  int* evict_fill;           // [2][NC]  survivors per key
  int* wave_buf;             // [3][TWKV_PREFILL_MAX_QUERIES]: sequence, row and position of a prefill call's queries, wave by wave
  int4* klist;               // [NT]  K tiles of the current decode call, widest class first: (tile, class | n_valid << 8, base block, query slot)
  int4* kpairs;              // [NT + 64]  the same list as items of two tiles of one class (entries 2 i, 2 i + 1) for the CTA-pair kernel;
                             //            a class with an odd number of tiles ends with a filler entry (.y bit 7 set)
  int* klist_count;          // [1]
  int* cta_start;            // [MAX_PLAN_CTAS + 1]  first list entry of every K-score CTA
  int* kv_link;              // [NT * 128]  K slot -> V slot of the same token, for the sequences of the current decode pass (rebuilt by every pass)
  int* vcut;                 // [query slots][n_splits + 1]  cut points of every sequence's V tile list into the splits of the V pass
  float* part_acc;           // [max_partials][Hq][d_kv]
  float* part_l;             // [max_partials][Hq]
  int4* gate_fix;            // rows the fused gate kernel hands to its fix-up kernel
  float* gate_scratch;       // COMPUTE mode logits: [GATE_PIECE][2][d_kv] (small calls) or one [128][d_kv] block per CTA (fused kernel)

  __host__ __device__ int4* desc(int l, int side) const { return tile_desc + ((size_t)l * 2 + side) * NT; }
  __host__ __device__ int* aux(int l, int side) const { return tile_aux + ((size_t)l * 2 + side) * NT * TILE; }
  __host__ __device__ unsigned short* rank(int l, int side) const { return tile_rank + ((size_t)l * 2 + side) * NT * TILE; }
  __host__ __device__ int* ntiles(int l) const { return n_tiles + l * 2; }
  __host__ __device__ int* fill_l(int l) const { return fill + (size_t)l * NK; }
  __host__ __device__ int* key_last_l(int l) const { return key_last + (size_t)l * NK; }
  __host__ __device__ int* kcc(int l) const { return kclass_count + l * NC; }
  __host__ __device__ int* kct(int l) const { return kclass_tiles + (size_t)l * NC * NT; }
  __host__ __device__ int* svc(int l) const { return seq_vcount + l * S; }
  __host__ __device__ int* svt(int l) const { return seq_vtiles + (size_t)l * S * TPS; }
  __host__ __device__ int* stok(int l) const { return seq_tokens + l * S; }
};

struct LayerParams {
  const void *Uinv_k, *Uinv_v, *W_k, *W_v;
  const float *b_k, *b_v;
};

// Order-preserving float <-> unsigned encoding so that atomicMax on unsigned is a float max.
// 0 encodes "nothing seen yet" (below every float, including -inf).
__host__ __device__ inline unsigned enc_ordered(float f) {
  unsigned b;
#ifdef __CUDA_ARCH__
  b = __float_as_uint(f);
#else
  union { float f; unsigned u; } c; c.f = f; b = c.u;
#endif
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ inline float dec_ordered(unsigned u) {
  if (u == 0u) return -INFINITY;
  unsigned b = (u & 0x80000000u) ? (u & 0x7fffffffu) : ~u;
  return __uint_as_float(b);
}

__device__ inline void set_status(const DevView& v, int code) { atomicCAS(v.status, 0, code); }

// The V pass walks a sequence's n V tiles in the order j -> (j * vtile_stride(n)) mod n: a stride near n / golden ratio,
// coprime to n, so that any run of consecutive j is spread evenly over the list.  Tiles of one class sit together in the
// list when a context was compressed in one call; a split that took a contiguous piece of the list itself would be all
// narrow or all wide tiles, and the narrow ones cost more per byte.
__device__ inline int vtile_stride(int n) {
  if (n < 3) return 1;
  int s = (int)(((long long)n * 618034ll) / 1000000ll);
  if (s < 1) s = 1;
  for (;; ++s) {
    int a = s, b = n;
    while (b) { const int t = a % b; a = b; b = t; }
    if (a == 1) return s;
  }
}

// Makes `dev` the current device for the scope of a host call.
struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    target = dev;
  }
  ~DeviceGuard() { if (prev >= 0 && prev != target) cudaSetDevice(prev); }
  int target = -1;
};

// launch bookkeeping (host)
void count_launch(int n = 1);
// optional per-kernel event timing of the cache whose API call is running on this thread
void prof_mark(int kind, cudaStream_t st, bool begin);
struct ProfScope {
  int kind; cudaStream_t st;
  ProfScope(int k, cudaStream_t s) : kind(k), st(s) { prof_mark(kind, st, true); }
  ~ProfScope() { prof_mark(kind, st, false); }
};

// kernels' host launchers (defined in the .cu files)
cudaError_t launch_rope_tables(const DevView& v, float rope_base, cudaStream_t st);
cudaError_t launch_clear_tables(const DevView& v, cudaStream_t st);
cudaError_t launch_gate_rank(const DevView& v, const float* logits, unsigned short* levels, int n_tok, cudaStream_t st);
cudaError_t launch_compress_pieces(const DevView& v, int layer, const void* K, const void* V, const int* seq_ids,
                                  const int* positions, int n_tok, const unsigned short* levels, cudaStream_t st);
struct TcMaps;   // tensor maps of the K-score kernel (api.cu)
cudaError_t launch_decode(const DevView& v, int layer, const LayerParams& lp, const void* q, const int* seq_ids,
                          int n_seq, void* out, int num_splits, int sm_count, const TcMaps* maps, bool pairs, cudaStream_t st);
struct GateMaps;   // tensor maps of the fused gate kernel (api.cu)
cudaError_t launch_gate_ranks_tc(const DevView& v, const GateMaps& maps, const LayerParams& lp, int n_tok, unsigned short* levels,
                                 int sm_count, bool pairs, cudaStream_t st);
int gate_tc_max_pairs(int sm_count);
size_t gate_tc_stage_bytes(int n_cta, int d);
size_t gate_tc_fix_bytes();
struct ProjectMaps;   // tensor maps of the projection kernel
cudaError_t launch_project_tc(const ProjectMaps& maps, int n_tok, int d, int bf16, int side0, int n_sides, int* status,
                              int sm_count, bool pairs, cudaStream_t st);
int project_tc_max_pairs(int sm_count);
cudaError_t launch_transpose16(const void* in, void* out, int n, cudaStream_t st);
cudaError_t launch_uinv_panels(const void* in, void* out, int d, cudaStream_t st);
int kscore_max_pairs(int sm_count);
cudaError_t launch_gate_logits(const DevView& v, const LayerParams& lp, const void* K, const void* V, int n_tok,
                               float* logits, cudaStream_t st);
cudaError_t launch_gate_soft(const DevView& v, const float* logits, const void* K, const void* V, float* mk, float* mv, float* xhk,
                             float* xhv, float* retain, int n_tok, cudaStream_t st);
cudaError_t launch_evict(const DevView& v, int layer, int seq, const int* keep_positions, int n_keep, cudaStream_t st);
cudaError_t launch_wait_timeout(const DevView& v, unsigned attempts, unsigned long long* out_dev, cudaStream_t st);
cudaError_t launch_cache_check(const DevView& v, int layer, const unsigned long long* guards_dev, int n_guards, unsigned long long* out_dev,
                               cudaStream_t st);
cudaError_t launch_stats(const DevView& v, int layer, unsigned long long* out_dev, cudaStream_t st);

}  // namespace twkv
