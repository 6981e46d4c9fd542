// C ABI of libtwkv: cache lifetime, argument checks, piece loop, launch bookkeeping.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <cudaTypedefs.h>

#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

struct Prof {
  bool on = false;
  std::vector<cudaEvent_t> ev;      // pairs: 2 * i = start, 2 * i + 1 = stop
  std::vector<int> kind;
  size_t used = 0;
  static constexpr size_t kMax = 8192;
};
static thread_local Prof* t_prof = nullptr;
void prof_mark(int kind, cudaStream_t st, bool begin) {
  Prof* p = t_prof;
  if (!p || !p->on) return;
  if (begin) {
    if (p->used >= Prof::kMax) return;
    p->kind[p->used] = kind;
    cudaEventRecord(p->ev[2 * p->used], st);
  } else {
    if (p->used >= Prof::kMax) return;
    cudaEventRecord(p->ev[2 * p->used + 1], st);
    ++p->used;
  }
}
struct ProfBind {
  explicit ProfBind(Prof* p) { t_prof = p; }
  ~ProfBind() { t_prof = nullptr; }
};

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
bool make_tmap_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_bytes, uint32_t box_rows) {
  static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
      cudaGetLastError();
      return false;
    }
    encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {row_stride_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)PANEL, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D tensor map over a row-major fp32 matrix [rows][cols], box [box_rows][box_cols], no swizzle.
static bool make_tmap_2d_f32(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
    cudaGetLastError();
    return false;
  }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * sizeof(float)};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn)(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides,
                                                                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Regions of the pool, each followed by one guard word (checked by twkv_cache_check).
struct Layout {
  size_t total = 0;
  std::vector<unsigned long long> guards;                  // byte offsets of the guard words
  bool guard = true;                                       // off while the tables that a reset clears in one sweep are laid out
  size_t alloc(size_t bytes, size_t align = 256) {
    total = (total + align - 1) / align * align;
    const size_t off = total;
    total += bytes;
    if (bytes && guard) {
      total = (total + 7) / 8 * 8;
      guards.push_back(total);
      total += 8;
    }
    return off;
  }
};

constexpr int GATE_PIECE = 8192;       // tokens per COMPUTE-mode gate piece (logits scratch rows)
constexpr int GATE_TC_MIN_TOKENS = 1024;   // calls at least this large run the fused tcgen05 gate kernel

struct Offsets {
  size_t status, pflags, rope_lo, rope_hi, n_tiles, tile_desc, tile_aux, tile_rank, fill, key_last, kclass_count,
      kclass_tiles, seq_vcount, seq_vtiles, seq_tokens, rank_sums, hist, key_cnt, key_old_fill, key_first_id,
      key_first_base, key_old_last, scores, seqmax, qslot, klist, kpairs, klist_count, cta_start, vcut, kv_link, wave_buf, evict_bitmap, evict_map, evict_fill, part_acc, part_l, gate_scratch, gate_fix, stats_buf, tables_end, prep_uinvT, prep_wT, guard_list,
      blocks, end_fixed;
};

struct Dims { int d_kv, NC, NT, TPS, NK, rep, max_partials, batch; };

static bool config_ok(const twkv_config* c) {
  if (!c) return false;
  if (c->head_dim != HEAD_DIM) return false;
  if (c->n_kv_heads < 1 || c->n_kv_heads > 8) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  const int rep = c->n_q_heads / c->n_kv_heads;
  if (!(rep == 1 || rep == 2 || rep == 4 || rep == 8)) return false;
  if (c->dtype != TWKV_F16 && c->dtype != TWKV_BF16) return false;
  if (c->out_dtype != TWKV_F16 && c->out_dtype != TWKV_BF16 && c->out_dtype != TWKV_F32) return false;
  if (c->n_layers < 1 || c->max_seqs < 1 || c->max_tokens_per_seq < 1) return false;
  if (c->max_seqs > 4096 || c->n_layers > 1024) return false;
  if ((long long)c->max_tokens_per_seq > (long long)ROPE_LO * ROPE_HI) return false;
  if (!(c->tau > 0.f && c->tau < 1.f)) return false;
  return true;
}

static Dims dims_of(const twkv_config* c) {
  Dims d;
  d.d_kv = c->n_kv_heads * c->head_dim;
  d.NC = d.d_kv / PANEL;
  d.TPS = (c->max_tokens_per_seq + TILE - 1) / TILE + d.NC;
  d.NT = c->max_seqs * d.TPS;
  d.NK = 2 * c->max_seqs * d.NC;
  d.rep = c->n_q_heads / c->n_kv_heads;
  d.max_partials = c->max_seqs + MAX_PARTIALS_EXTRA;
  // pieces whose bookkeeping kernels are launched together: up to 4, while their chunk-count tables stay under 64 MiB
  const size_t hist_piece = (size_t)PIECE_CHUNKS * d.NK * sizeof(int);
  d.batch = (int)((size_t)(64u << 20) / hist_piece);
  if (d.batch < 1) d.batch = 1;
  if (d.batch > 4) d.batch = 4;
  return d;
}

static Offsets layout_of(const twkv_config* c, const Dims& d, std::vector<unsigned long long>* guards = nullptr) {
  Layout L;
  Offsets o;
  const size_t Ls = c->n_layers, S = c->max_seqs, NT = d.NT, NK = d.NK, Hq = c->n_q_heads;
  o.status = L.alloc(8 * sizeof(int));
  o.rope_lo = L.alloc((size_t)ROPE_LO * 32 * sizeof(float4));
  o.rope_hi = L.alloc((size_t)ROPE_HI * 32 * sizeof(float4));
  L.guard = false;
  o.n_tiles = L.alloc(Ls * 2 * sizeof(int));
  o.tile_desc = L.alloc(Ls * 2 * NT * sizeof(int4));
  o.tile_aux = L.alloc(Ls * 2 * NT * TILE * sizeof(int));
  o.tile_rank = L.alloc(Ls * 2 * NT * TILE * sizeof(unsigned short));
  o.fill = L.alloc(Ls * NK * sizeof(int));
  o.key_last = L.alloc(Ls * NK * sizeof(int));
  o.kclass_count = L.alloc(Ls * d.NC * sizeof(int));
  o.kclass_tiles = L.alloc(Ls * d.NC * NT * sizeof(int));
  o.seq_vcount = L.alloc(Ls * S * sizeof(int));
  o.seq_vtiles = L.alloc(Ls * S * d.TPS * sizeof(int));
  o.seq_tokens = L.alloc(Ls * S * sizeof(int));
  o.rank_sums = L.alloc(Ls * 2 * sizeof(unsigned long long));
  o.tables_end = L.alloc(0);
  L.guard = true;
  L.alloc(8);                                              // one guard behind the tables
  const size_t PB = (size_t)d.batch;
  o.hist = L.alloc(PB * PIECE_CHUNKS * NK * sizeof(int));
  o.key_cnt = L.alloc(PB * NK * sizeof(int));
  o.key_old_fill = L.alloc(PB * NK * sizeof(int));
  o.key_first_id = L.alloc(PB * NK * sizeof(int));
  o.key_first_base = L.alloc(PB * NK * sizeof(int));
  o.key_old_last = L.alloc(PB * NK * sizeof(int));
  o.pflags = L.alloc(PB * 2 * sizeof(int));
  o.scores = L.alloc(NT * TILE * Hq * sizeof(float));
  o.seqmax = L.alloc(S * Hq * sizeof(unsigned));
  o.qslot = L.alloc(S * sizeof(int));
  o.klist = L.alloc(NT * sizeof(int4));
  o.klist_count = L.alloc(sizeof(int));
  o.kpairs = L.alloc((NT + 64) * sizeof(int4));
  o.cta_start = L.alloc((MAX_PLAN_CTAS + 1) * sizeof(int));
  o.vcut = L.alloc((size_t)(d.max_partials + S + 1) * sizeof(int));
  o.kv_link = L.alloc((size_t)NT * TILE * sizeof(int));
  o.wave_buf = L.alloc((size_t)3 * TWKV_PREFILL_MAX_QUERIES * sizeof(int));
  o.evict_bitmap = L.alloc((size_t)ROPE_LO * ROPE_HI / 8);
  o.evict_map = L.alloc((size_t)2 * NT * TILE * sizeof(int));
  o.evict_fill = L.alloc((size_t)2 * d.NC * sizeof(int));
  o.part_acc = L.alloc((size_t)d.max_partials * Hq * d.d_kv * sizeof(float));
  o.part_l = L.alloc((size_t)d.max_partials * Hq * sizeof(float));
  {
    const size_t small = (size_t)GATE_PIECE * 2 * d.d_kv * sizeof(float), fused = gate_tc_stage_bytes(MAX_PLAN_CTAS < 160 ? MAX_PLAN_CTAS : 160, d.d_kv);
    o.gate_scratch = L.alloc(small > fused ? small : fused);
  }
  o.gate_fix = L.alloc(gate_tc_fix_bytes());
  o.stats_buf = L.alloc(64 * sizeof(unsigned long long));
  o.prep_uinvT = L.alloc(Ls * (size_t)d.d_kv * d.d_kv * 2, 1024);
  o.prep_wT = L.alloc(Ls * 2 * (size_t)d.d_kv * d.d_kv * 2, 1024);
  o.guard_list = L.alloc(L.guards.size() * sizeof(unsigned long long) + 64);
  o.blocks = L.alloc(0, 1024);
  o.end_fixed = o.blocks;
  if (guards) *guards = L.guards;
  return o;
}

}  // namespace twkv

using namespace twkv;

struct twkv_cache {
  twkv_config cfg;
  Dims dims;
  Offsets off;
  DevView view;
  unsigned char* pool;
  size_t pool_bytes;
  int device;
  int sm_count;
  std::vector<LayerParams> params;
  Prof prof;
  CUtensorMap map_blocks;
  CUtensorMap map_scores;              // the score scratch as [V slot][Hq] fp32, boxes of one tile's rows x one V-pass CTA's heads
  bool scores_tma = false;             // the head count allows that map (rows must start on 16-byte boundaries)
  std::vector<CUtensorMap> map_uinvT;  // per layer, over the transposed copy of U_K^-1 inside the pool
  std::vector<char> prepared;          // per layer: transposed copy and its map are current
  std::vector<CUtensorMap> map_wT;     // per layer x side, over the transposed copies of the gate weights (box = one slab)
  std::vector<CUtensorMap> map_wT_half; // the same with 128-row boxes, for the CTA-pair kernel
  std::vector<char> prepared_w;        // per layer: those copies and maps are current
  bool kscore_pairs = false;           // the K-score kernel runs on CTA pairs (the device can co-schedule them)
  std::vector<unsigned long long> guards;   // byte offsets (from the pool's start) of the guard words
};


extern "C" {

const char* twkv_status_string(twkv_status s) {
  switch (s) {
    case TWKV_OK: return "ok";
    case TWKV_ERR_INVALID_ARG: return "invalid argument";
    case TWKV_ERR_UNSUPPORTED: return "unsupported configuration";
    case TWKV_ERR_CAPACITY: return "cache capacity exhausted";
    case TWKV_ERR_CUDA: return "CUDA runtime error";
    case TWKV_ERR_DEVICE_CHECK: return "device-side check failed";
    case TWKV_ERR_TIMEOUT: return "bounded device wait timed out";
  }
  return "unknown status";
}

uint64_t twkv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t twkv_cache_required_bytes(const twkv_config* cfg, size_t payload_bytes) {
  if (!config_ok(cfg)) return 0;
  const Dims d = dims_of(cfg);
  const Offsets o = layout_of(cfg, d);
  // every (layer, sequence, side) may hold one partially filled tile of every class
  const size_t slack_blocks = (size_t)cfg->n_layers * cfg->max_seqs * 2 * ((size_t)d.NC * (d.NC + 1) / 2);
  const size_t payload_blocks = (payload_bytes + BLOCK_BYTES - 1) / BLOCK_BYTES;
  return o.blocks + (payload_blocks + slack_blocks) * (size_t)BLOCK_BYTES;
}

static void fill_view(twkv_cache* c) {
  DevView& v = c->view;
  const twkv_config& cfg = c->cfg;
  const Dims& d = c->dims;
  const Offsets& o = c->off;
  unsigned char* p = c->pool;
  v.L = cfg.n_layers; v.Hq = cfg.n_q_heads; v.Hkv = cfg.n_kv_heads; v.rep = d.rep; v.d_kv = d.d_kv; v.NC = d.NC;
  v.S = cfg.max_seqs; v.tmax = cfg.max_tokens_per_seq; v.NT = d.NT; v.TPS = d.TPS; v.dtype = cfg.dtype;
  v.out_dtype = cfg.out_dtype; v.NK = d.NK; v.max_partials = d.max_partials; v.tau = cfg.tau; v.sm_scale = cfg.sm_scale;
  const size_t nb = (c->pool_bytes - o.blocks) / BLOCK_BYTES;
  v.n_blocks = (int)(nb > 0x7fffffffull ? 0x7fffffffull : nb);
  v.status = (int*)(p + o.status); v.pflags = (int*)(p + o.pflags); v.batch = d.batch;
  v.rope_lo = (float4*)(p + o.rope_lo); v.rope_hi = (float4*)(p + o.rope_hi);
  v.blocks = p + o.blocks;
  v.n_tiles = (int*)(p + o.n_tiles); v.tile_desc = (int4*)(p + o.tile_desc); v.tile_aux = (int*)(p + o.tile_aux);
  v.tile_rank = (unsigned short*)(p + o.tile_rank); v.fill = (int*)(p + o.fill); v.key_last = (int*)(p + o.key_last);
  v.kclass_count = (int*)(p + o.kclass_count); v.kclass_tiles = (int*)(p + o.kclass_tiles);
  v.seq_vcount = (int*)(p + o.seq_vcount); v.seq_vtiles = (int*)(p + o.seq_vtiles); v.seq_tokens = (int*)(p + o.seq_tokens);
  v.rank_sums = (unsigned long long*)(p + o.rank_sums);
  v.hist = (int*)(p + o.hist); v.key_cnt = (int*)(p + o.key_cnt); v.key_old_fill = (int*)(p + o.key_old_fill);
  v.key_first_id = (int*)(p + o.key_first_id); v.key_first_base = (int*)(p + o.key_first_base);
  v.key_old_last = (int*)(p + o.key_old_last);
  v.scores = (float*)(p + o.scores); v.seqmax = (unsigned*)(p + o.seqmax); v.qslot = (int*)(p + o.qslot);
  v.klist = (int4*)(p + o.klist); v.klist_count = (int*)(p + o.klist_count);
  v.kpairs = (int4*)(p + o.kpairs); v.cta_start = (int*)(p + o.cta_start); v.vcut = (int*)(p + o.vcut); v.kv_link = (int*)(p + o.kv_link);
  v.part_acc = (float*)(p + o.part_acc); v.part_l = (float*)(p + o.part_l);
  v.gate_scratch = (float*)(p + o.gate_scratch);
  v.gate_fix = (int4*)(p + o.gate_fix);
  v.wave_buf = (int*)(p + o.wave_buf);
  v.evict_bitmap = (unsigned*)(p + o.evict_bitmap); v.evict_map = (int*)(p + o.evict_map); v.evict_fill = (int*)(p + o.evict_fill);
  v.qmap = nullptr; v.qpos = nullptr;
}

twkv_status twkv_cache_reset(twkv_cache* c, void* stream) {
  if (!c) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  // every table between the RoPE tables and the scratch starts from zero; key_last from -1
  if (cudaMemsetAsync(c->pool + c->off.n_tiles, 0, c->off.tables_end - c->off.n_tiles, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (cudaMemsetAsync(c->pool + c->off.key_last, 0xff, (size_t)c->cfg.n_layers * c->dims.NK * sizeof(int), st) != cudaSuccess)
    return TWKV_ERR_CUDA;
  if (cudaMemsetAsync(c->pool + c->off.status, 0, 8 * sizeof(int), st) != cudaSuccess) return TWKV_ERR_CUDA;
  return TWKV_OK;
}

twkv_status twkv_cache_create(const twkv_config* cfg, void* pool, size_t pool_bytes, void* stream, twkv_cache** out) {
  if (!cfg || !pool || !out) return TWKV_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg)) return TWKV_ERR_UNSUPPORTED;
  if ((uintptr_t)pool % 256) return TWKV_ERR_INVALID_ARG;
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, pool) != cudaSuccess) { cudaGetLastError(); return TWKV_ERR_CUDA; }
  if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) return TWKV_ERR_INVALID_ARG;
  const Dims d = dims_of(cfg);
  std::vector<unsigned long long> guards;
  const Offsets o = layout_of(cfg, d, &guards);
  if (pool_bytes < o.blocks + (size_t)BLOCK_BYTES) return TWKV_ERR_CAPACITY;
  twkv_cache* c = new (std::nothrow) twkv_cache();
  if (!c) return TWKV_ERR_INVALID_ARG;
  c->guards = guards;
  c->cfg = *cfg; c->dims = d; c->off = o; c->pool = (unsigned char*)pool; c->pool_bytes = pool_bytes;
  c->device = attr.device;
  c->params.assign(cfg->n_layers, LayerParams{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr});
  DeviceGuard g(c->device);
  if (!g.ok) { delete c; return TWKV_ERR_CUDA; }
  if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) { delete c; return TWKV_ERR_CUDA; }
  if (c->sm_count > MAX_PLAN_CTAS) c->sm_count = MAX_PLAN_CTAS;
  {
    // TWKV_KSCORE_SINGLE=1 keeps the K-score kernel on single CTAs (the fallback where CTA pairs cannot be scheduled)
    const char* single = getenv("TWKV_KSCORE_SINGLE");
    c->kscore_pairs = !(single && single[0] == '1') && kscore_max_pairs(c->sm_count) > 0;
  }
  fill_view(c);
  {
    const char* dbg = getenv("TWKV_DEBUG");
    c->view.debug = (dbg && dbg[0] == '1') ? 1 : 0;
  }
  c->map_uinvT.resize(cfg->n_layers);
  c->prepared.assign(cfg->n_layers, 0);
  c->map_wT.resize(2 * (size_t)cfg->n_layers);
  c->map_wT_half.resize(2 * (size_t)cfg->n_layers);
  c->prepared_w.assign(cfg->n_layers, 0);
  if (!make_tmap_2d(&c->map_blocks, c->view.blocks, (uint64_t)c->view.n_blocks * TILE, PANEL, PANEL * 2, TILE)) { delete c; return TWKV_ERR_CUDA; }
  if (c->cfg.n_q_heads % 4 == 0) {
    const int hq = c->cfg.n_q_heads, nb = hq < 16 ? hq : (hq <= 16 ? 16 : 32);
    if (!make_tmap_2d_f32(&c->map_scores, c->view.scores, (uint64_t)c->dims.NT * TILE, (uint64_t)hq, TILE, (uint32_t)(nb < hq ? nb : hq))) { delete c; return TWKV_ERR_CUDA; }
    c->scores_tma = true;
  }
  {
    // guard words behind every region, and the list of their offsets for the check kernel
    const unsigned long long word = TWKV_GUARD_WORD;
    for (unsigned long long off : c->guards)
      if (cudaMemcpyAsync(c->pool + off, &word, sizeof(word), cudaMemcpyHostToDevice, (cudaStream_t)stream) != cudaSuccess) { delete c; return TWKV_ERR_CUDA; }
    if (cudaMemcpyAsync(c->pool + o.guard_list, c->guards.data(), c->guards.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice,
                        (cudaStream_t)stream) != cudaSuccess) { delete c; return TWKV_ERR_CUDA; }
  }
  twkv_status s = twkv_cache_reset(c, stream);
  if (s != TWKV_OK) { delete c; return s; }
  if (launch_rope_tables(c->view, cfg->rope_base, (cudaStream_t)stream) != cudaSuccess) { delete c; return TWKV_ERR_CUDA; }
  *out = c;
  return TWKV_OK;
}

twkv_status twkv_profile_enable(twkv_cache* c, int enable) {
  if (!c) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  Prof& p = c->prof;
  if (enable && p.ev.empty()) {
    p.ev.resize(2 * Prof::kMax);
    p.kind.assign(Prof::kMax, 0);
    for (auto& e : p.ev)
      if (cudaEventCreate(&e) != cudaSuccess) return TWKV_ERR_CUDA;
  }
  p.on = enable != 0;
  p.used = 0;
  return TWKV_OK;
}

twkv_status twkv_profile_read(twkv_cache* c, void* stream, double* ms, uint64_t* launches) {
  if (!c || !ms || !launches) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return TWKV_ERR_CUDA;
  for (int k = 0; k < TWKV_N_KERNELS; ++k) { ms[k] = 0.0; launches[k] = 0; }
  Prof& p = c->prof;
  for (size_t i = 0; i < p.used; ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, p.ev[2 * i], p.ev[2 * i + 1]) != cudaSuccess) return TWKV_ERR_CUDA;
    ms[p.kind[i]] += (double)t;
    launches[p.kind[i]] += 1;
  }
  p.used = 0;
  return TWKV_OK;
}

twkv_status twkv_cache_destroy(twkv_cache* c) {
  if (!c) return TWKV_ERR_INVALID_ARG;
  for (auto& e : c->prof.ev) cudaEventDestroy(e);
  delete c;
  return TWKV_OK;
}

twkv_status twkv_cache_set_layer_params(twkv_cache* c, int layer, const twkv_layer_params* p) {
  if (!c || !p || layer < 0 || layer >= c->cfg.n_layers) return TWKV_ERR_INVALID_ARG;
  if (!p->Uinv_k || !p->Uinv_v) return TWKV_ERR_INVALID_ARG;
  if (((uintptr_t)p->Uinv_k | (uintptr_t)p->Uinv_v | (uintptr_t)p->W_k | (uintptr_t)p->W_v | (uintptr_t)p->b_k | (uintptr_t)p->b_v) % 16) return TWKV_ERR_INVALID_ARG;
  c->params[layer] = LayerParams{p->Uinv_k, p->Uinv_v, p->W_k, p->W_v, p->b_k, p->b_v};
  c->prepared[layer] = 0;
  c->prepared_w[layer] = 0;
  return TWKV_OK;
}

twkv_status twkv_compress(twkv_cache* c, int layer, const void* K, const void* V, const int32_t* seq_ids,
                          const int32_t* positions, int n_tok, const float* scores, uint16_t* levels,
                          twkv_gate_mode mode, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || n_tok < 0) return TWKV_ERR_INVALID_ARG;
  if (n_tok == 0) return TWKV_OK;
  if (!K || !V || !seq_ids || !positions || !levels) return TWKV_ERR_INVALID_ARG;
  if (((uintptr_t)K | (uintptr_t)V) % 16 || (uintptr_t)levels % 4) return TWKV_ERR_INVALID_ARG;
  if (mode == TWKV_GATE_LOGITS && (!scores || (uintptr_t)scores % 16)) return TWKV_ERR_INVALID_ARG;
  if (mode == TWKV_GATE_COMPUTE && (!c->params[layer].W_k || !c->params[layer].W_v)) return TWKV_ERR_INVALID_ARG;
  if (mode != TWKV_GATE_FORCED && mode != TWKV_GATE_LOGITS && mode != TWKV_GATE_COMPUTE) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  ProfBind pb(&c->prof);
  cudaStream_t st = (cudaStream_t)stream;
  const DevView& v = c->view;
  const size_t row = (size_t)v.d_kv * 2;
  if (mode == TWKV_GATE_LOGITS) {
    if (launch_gate_rank(v, scores, levels, n_tok, st) != cudaSuccess) return TWKV_ERR_CUDA;
  } else if (mode == TWKV_GATE_COMPUTE && n_tok >= GATE_TC_MIN_TOKENS && c->sm_count <= 160) {
    // fused tcgen05 kernel: logits and ranks in one launch, the logits never leave the CTA's staging block
    const int d = c->dims.d_kv;
    if (!c->prepared_w[layer]) {
      // first COMPUTE call after the parameters were (re)set: K-major copies of W_k, W_v for the tensor cores
      const int ns = (d % 256 == 0) ? 256 : 128;
      for (int side = 0; side < 2; ++side) {
        unsigned char* dst = c->pool + c->off.prep_wT + ((size_t)layer * 2 + side) * d * d * 2;
        if (launch_transpose16(side ? c->params[layer].W_v : c->params[layer].W_k, dst, d, st) != cudaSuccess) return TWKV_ERR_CUDA;
        if (!make_tmap_2d(&c->map_wT[2 * (size_t)layer + side], dst, d, d, (uint64_t)d * 2, ns) ||
            !make_tmap_2d(&c->map_wT_half[2 * (size_t)layer + side], dst, d, d, (uint64_t)d * 2, TILE)) return TWKV_ERR_CUDA;
      }
      c->prepared_w[layer] = 1;
    }
    const bool pairs = d % 256 == 0 && gate_tc_max_pairs(c->sm_count) > 0;
    GateMaps maps;
    maps.wk = (pairs ? c->map_wT_half : c->map_wT)[2 * (size_t)layer];
    maps.wv = (pairs ? c->map_wT_half : c->map_wT)[2 * (size_t)layer + 1];
    if (!make_tmap_2d(&maps.xk, K, (uint64_t)n_tok, d, (uint64_t)d * 2, TILE) ||
        !make_tmap_2d(&maps.xv, V, (uint64_t)n_tok, d, (uint64_t)d * 2, TILE)) return TWKV_ERR_CUDA;
    const unsigned char* wT = c->pool + c->off.prep_wT + (size_t)layer * 2 * d * d * 2;
    maps.raw = GateRaw{(const unsigned short*)K, (const unsigned short*)V, (const unsigned short*)wT,
                       (const unsigned short*)(wT + (size_t)d * d * 2), v.gate_fix, v.status + 2};
    if (launch_gate_ranks_tc(v, maps, c->params[layer], n_tok, levels, c->sm_count, pairs, st) != cudaSuccess) return TWKV_ERR_CUDA;
  } else if (mode == TWKV_GATE_COMPUTE) {
    for (int lo = 0; lo < n_tok; lo += GATE_PIECE) {
      const int n = n_tok - lo < GATE_PIECE ? n_tok - lo : GATE_PIECE;
      if (launch_gate_logits(v, c->params[layer], (const unsigned char*)K + lo * row, (const unsigned char*)V + lo * row, n,
                             v.gate_scratch, st) != cudaSuccess) return TWKV_ERR_CUDA;
      if (launch_gate_rank(v, v.gate_scratch, levels + 2 * (size_t)lo, n, st) != cudaSuccess) return TWKV_ERR_CUDA;
    }
  }
  const int group = TWKV_PIECE_TOKENS * c->dims.batch;     // tokens whose pieces are handled by one set of launches
  for (int lo = 0; lo < n_tok; lo += group) {
    const int n = n_tok - lo < group ? n_tok - lo : group;
    if (launch_compress_pieces(v, layer, (const unsigned char*)K + lo * row, (const unsigned char*)V + lo * row, seq_ids + lo,
                               positions + lo, n, levels + 2 * (size_t)lo, st) != cudaSuccess) return TWKV_ERR_CUDA;
  }
  return TWKV_OK;
}

// One pass of the decode kernels: one query per listed sequence.  qmap / qpos (device, per query slot) are set for a
// prefill wave: the row of q / out a slot stands for, and the last position it may attend to.
static twkv_status decode_pass(twkv_cache* c, int layer, const void* q, const int32_t* seq_ids, int n_seq, void* out,
                               int num_splits, const int* qmap, const int* qpos, cudaStream_t stream) {
  if (n_seq > c->cfg.max_seqs) return TWKV_ERR_INVALID_ARG;
  if (!c->params[layer].Uinv_k || !c->params[layer].Uinv_v) return TWKV_ERR_INVALID_ARG;
  const int head_groups = (c->cfg.n_q_heads + 31) / 32;
  if (num_splits == 0) {
    num_splits = c->sm_count / (n_seq * head_groups);
    if (num_splits < 1) num_splits = 1;
    if (num_splits > 64) num_splits = 64;
  }
  if ((long long)n_seq * num_splits > c->dims.max_partials) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  ProfBind pb(&c->prof);
  if (!c->prepared[layer]) {
    // first decode after the parameters were (re)set: U_K^-1 re-tiled into the contiguous K-major panels the tensor cores read
    unsigned char* dst = c->pool + c->off.prep_uinvT + (size_t)layer * c->dims.d_kv * c->dims.d_kv * 2;
    if (launch_uinv_panels(c->params[layer].Uinv_k, dst, c->dims.d_kv, (cudaStream_t)stream) != cudaSuccess) return TWKV_ERR_CUDA;
    // box = a whole panel for the single-CTA kernel, the CTA's half of its rows for the pair kernel
    if (!make_tmap_2d(&c->map_uinvT[layer], dst, (uint64_t)c->dims.NC * c->dims.d_kv, PANEL, PANEL * 2,
                      c->kscore_pairs ? HEAD_DIM / 2 : HEAD_DIM)) return TWKV_ERR_CUDA;
    c->prepared[layer] = 1;
  }
  TcMaps maps;
  maps.blocks = c->map_blocks;
  maps.scores = c->scores_tma ? &c->map_scores : nullptr;
  maps.uinvT_k = c->map_uinvT[layer];
  DevView v = c->view;
  v.qmap = qmap; v.qpos = qpos;
  if (launch_decode(v, layer, c->params[layer], q, seq_ids, n_seq, out, num_splits, c->sm_count, &maps, c->kscore_pairs,
                    (cudaStream_t)stream) != cudaSuccess) return TWKV_ERR_CUDA;
  return TWKV_OK;
}

twkv_status twkv_decode_attn(twkv_cache* c, int layer, const void* q, const int32_t* seq_ids, int n_seq, void* out,
                             int num_splits, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || n_seq < 0 || num_splits < 0) return TWKV_ERR_INVALID_ARG;
  if (n_seq == 0) return TWKV_OK;
  if (!q || !seq_ids || !out || n_seq > c->cfg.max_seqs) return TWKV_ERR_INVALID_ARG;
  if (((uintptr_t)q | (uintptr_t)out) % 16) return TWKV_ERR_INVALID_ARG;
  return decode_pass(c, layer, q, seq_ids, n_seq, out, num_splits, nullptr, nullptr, (cudaStream_t)stream);
}

twkv_status twkv_prefill_attn(twkv_cache* c, int layer, const void* q, const int32_t* q_seq, const int32_t* q_pos, int n_q,
                              void* out, int num_splits, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || n_q < 0 || num_splits < 0) return TWKV_ERR_INVALID_ARG;
  if (n_q == 0) return TWKV_OK;
  if (!q || !q_seq || !q_pos || !out || n_q > TWKV_PREFILL_MAX_QUERIES) return TWKV_ERR_INVALID_ARG;
  if (((uintptr_t)q | (uintptr_t)out) % 16) return TWKV_ERR_INVALID_ARG;
  const int S = c->cfg.max_seqs;
  // wave k = the k-th query of every sequence, in order of appearance; inside a wave the sequences are distinct
  std::vector<int> seen(S, 0), wave_of(n_q);
  int n_waves = 0;
  for (int i = 0; i < n_q; ++i) {
    if (q_seq[i] < 0 || q_seq[i] >= S || q_pos[i] < 0) return TWKV_ERR_INVALID_ARG;
    wave_of[i] = seen[q_seq[i]]++;
    if (wave_of[i] + 1 > n_waves) n_waves = wave_of[i] + 1;
  }
  std::vector<int> wave_start(n_waves + 1, 0), fill(n_waves, 0);
  for (int i = 0; i < n_q; ++i) ++wave_start[wave_of[i] + 1];
  for (int w = 0; w < n_waves; ++w) wave_start[w + 1] += wave_start[w];
  std::vector<int> host(3 * (size_t)TWKV_PREFILL_MAX_QUERIES);
  for (int i = 0; i < n_q; ++i) {
    const int at = wave_start[wave_of[i]] + fill[wave_of[i]]++;
    host[at] = q_seq[i];
    host[TWKV_PREFILL_MAX_QUERIES + at] = i;
    host[2 * TWKV_PREFILL_MAX_QUERIES + at] = q_pos[i];
  }
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  // the copy is staged from pageable memory before the call returns, so `host` may go out of scope afterwards
  if (cudaMemcpyAsync(c->view.wave_buf, host.data(), host.size() * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess) return TWKV_ERR_CUDA;
  for (int w = 0; w < n_waves; ++w) {
    const int off = wave_start[w], n = wave_start[w + 1] - off;
    twkv_status s = decode_pass(c, layer, q, c->view.wave_buf + off, n, out, num_splits, c->view.wave_buf + TWKV_PREFILL_MAX_QUERIES + off,
                                c->view.wave_buf + 2 * TWKV_PREFILL_MAX_QUERIES + off, st);
    if (s != TWKV_OK) return s;
  }
  return TWKV_OK;
}

twkv_status twkv_cache_status(twkv_cache* c, void* stream) {
  if (!c) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  int code = 0;
  if (cudaMemcpyAsync(&code, c->view.status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (code != 0) {
    if (cudaMemsetAsync(c->view.status, 0, sizeof(int), st) != cudaSuccess) return TWKV_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  }
  return (twkv_status)code;
}

twkv_status twkv_cache_check(twkv_cache* c, int layer, void* stream, uint64_t* violations) {
  if (!c || layer < -1 || layer >= c->cfg.n_layers) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned long long* dev = (unsigned long long*)(c->pool + c->off.stats_buf);
  // guard offsets are relative to the pool; the kernel addresses them from the status word, which sits at its start
  if (launch_cache_check(c->view, layer, (const unsigned long long*)(c->pool + c->off.guard_list), (int)c->guards.size(), dev, st) != cudaSuccess)
    return TWKV_ERR_CUDA;
  unsigned long long bad = 0;
  if (cudaMemcpyAsync(&bad, dev, sizeof(bad), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (violations) *violations = bad;
  return bad ? TWKV_ERR_DEVICE_CHECK : TWKV_OK;
}

twkv_status twkv_selftest_wait_timeout(twkv_cache* c, uint32_t attempts, uint64_t* elapsed_ns, void* stream) {
  if (!c || attempts == 0) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned long long* dev = (unsigned long long*)(c->pool + c->off.stats_buf);
  if (launch_wait_timeout(c->view, attempts, dev, st) != cudaSuccess) return TWKV_ERR_CUDA;
  unsigned long long h[3] = {0, 0, 0};
  if (cudaMemcpyAsync(h, dev, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (elapsed_ns) *elapsed_ns = h[0];
  return (h[1] == 1 && h[2] == 1) ? TWKV_OK : TWKV_ERR_DEVICE_CHECK;     // the wait must have failed and raised the flag
}

twkv_status twkv_evict(twkv_cache* c, int layer, int seq, const int32_t* keep_positions, int n_keep, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || seq < 0 || seq >= c->cfg.max_seqs || n_keep < 0) return TWKV_ERR_INVALID_ARG;
  if (n_keep > 0 && !keep_positions) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  ProfBind pb(&c->prof);
  if (launch_evict(c->view, layer, seq, keep_positions, n_keep, (cudaStream_t)stream) != cudaSuccess) return TWKV_ERR_CUDA;
  return TWKV_OK;
}

twkv_status twkv_gate_soft(twkv_cache* c, int layer, const void* K, const void* V, int n_tok, float* m_k, float* m_v, float* xh_k,
                           float* xh_v, float* retain, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || n_tok < 0) return TWKV_ERR_INVALID_ARG;
  if (n_tok == 0) return TWKV_OK;
  if (!K || !V || ((uintptr_t)K | (uintptr_t)V) % 16) return TWKV_ERR_INVALID_ARG;
  if (!c->params[layer].W_k || !c->params[layer].W_v) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  ProfBind pb(&c->prof);
  cudaStream_t st = (cudaStream_t)stream;
  const DevView& v = c->view;
  const size_t row = (size_t)v.d_kv * 2, d = (size_t)v.d_kv;
  for (int lo = 0; lo < n_tok; lo += GATE_PIECE) {               // the logits of a piece live in the gate scratch
    const int n = n_tok - lo < GATE_PIECE ? n_tok - lo : GATE_PIECE;
    const unsigned char* kp = (const unsigned char*)K + lo * row;
    const unsigned char* vp = (const unsigned char*)V + lo * row;
    if (launch_gate_logits(v, c->params[layer], kp, vp, n, v.gate_scratch, st) != cudaSuccess) return TWKV_ERR_CUDA;
    if (launch_gate_soft(v, v.gate_scratch, kp, vp, m_k ? m_k + lo * d : nullptr, m_v ? m_v + lo * d : nullptr,
                         xh_k ? xh_k + lo * d : nullptr, xh_v ? xh_v + lo * d : nullptr, retain ? retain + 2 * (size_t)lo : nullptr, n,
                         st) != cudaSuccess) return TWKV_ERR_CUDA;
  }
  return TWKV_OK;
}

twkv_status twkv_cache_stats(twkv_cache* c, int layer, void* stream, twkv_stats* out) {
  if (!c || !out || layer < -1 || layer >= c->cfg.n_layers) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned long long* dev = (unsigned long long*)(c->pool + c->off.stats_buf);
  if (launch_stats(c->view, layer, dev, st) != cudaSuccess) return TWKV_ERR_CUDA;
  unsigned long long h[5 + 2 * TWKV_MAX_CLASSES];
  if (cudaMemcpyAsync(h, dev, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  memset(out, 0, sizeof(*out));
  out->tokens = h[0];
  out->bytes_stored = h[1];
  out->bytes_algorithmic = 2 * (h[2] + h[3]);
  out->blocks_used = h[4];
  out->blocks_free = (unsigned long long)c->view.n_blocks - h[4];
  const double denom = (double)h[0] * c->dims.d_kv;
  out->retain_rate_k = h[0] ? (double)h[2] / denom : 0.0;
  out->retain_rate_v = h[0] ? (double)h[3] / denom : 0.0;
  for (int s = 0; s < 2; ++s)
    for (int k = 0; k < TWKV_MAX_CLASSES; ++k) out->tokens_per_class[s][k] = h[5 + s * TWKV_MAX_CLASSES + k];
  return TWKV_OK;
}

twkv_status twkv_cache_layout(const twkv_cache* c, twkv_layout* out) {
  if (!c || !out) return TWKV_ERR_INVALID_ARG;
  const Offsets& o = c->off;
  out->pool_bytes = c->pool_bytes; out->n_blocks = (uint64_t)c->view.n_blocks; out->blocks_off = o.blocks;
  out->status_off = o.status; out->n_tiles_off = o.n_tiles; out->tile_desc_off = o.tile_desc; out->tile_aux_off = o.tile_aux;
  out->tile_rank_off = o.tile_rank; out->fill_off = o.fill; out->kclass_count_off = o.kclass_count;
  out->kclass_tiles_off = o.kclass_tiles; out->seq_vcount_off = o.seq_vcount; out->seq_vtiles_off = o.seq_vtiles;
  out->seq_tokens_off = o.seq_tokens; out->max_tiles = (uint64_t)c->dims.NT; out->tiles_per_seq = (uint64_t)c->dims.TPS;
  out->n_classes = (uint64_t)c->dims.NC;
  return TWKV_OK;
}

}  // extern "C"
