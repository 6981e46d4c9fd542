/*
 * libtwkv — token-wise adaptive low-rank KV-cache compression on one B200 (sm_100a).
 *
 * The method (Sec. 3 of the paper): a token's pre-RoPE key and value states are
 * expressed in a spectral basis, x~ = x U (Eq. 1).  A learned gate decides per
 * token, per layer and separately for K and V how many leading components to
 * keep (Eq. 5, Eq. 6, Eq. 8); only those r components are persisted (Eq. 2).
 * At decode time the states are rebuilt as x^[I] U^-1[I,:] (Eq. 3), keys are
 * reshaped to heads and rotated (RoPE), and ordinary softmax attention runs
 * over them.  The per-token "compression level" is the retained rank r.
 *
 * This library is the data-parallel hot path of that method:
 *   twkv_compress     gate -> rank -> truncate -> pack into a rank-class-sorted paged cache
 *   twkv_decode_attn  attention of one query per sequence over the mixed-rank cache
 *
 * Conventions
 *   - Every pointer argument is a DEVICE pointer unless its comment says "host".
 *   - The caller owns all device memory: inputs, outputs, layer parameters
 *     (borrowed until the cache is destroyed or the parameters are replaced)
 *     and the one `pool` buffer the cache lives in.  The library allocates no
 *     device memory; it allocates small host structures only.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream) and is asynchronous unless stated otherwise.  All scratch
 *     (scores, work lists, partial sums, gate staging) lives in the cache's one
 *     pool and is shared by its layers: calls on one cache must be ordered, on
 *     one stream or by events; calls that overlap on the GPU race.
 *   - Errors are return codes, never aborts.  Argument errors that the host can
 *     see are returned before anything is launched and leave the cache
 *     unchanged.  Errors only the device can see (pool exhausted, a rank or
 *     sequence id out of range) set a sticky status word; the offending piece
 *     of work is skipped as a whole (a decode query whose sequence id is out of
 *     range gets zeros) and the code is returned by the next
 *     twkv_cache_status().
 *   - Supported shapes: head_dim = 128, 1..8 KV heads (d_kv = n_kv_heads * 128,
 *     at most 1024), n_q_heads / n_kv_heads in {1, 2, 4, 8}.
 *
 * Cache container (the paper only fixes WHAT is stored, the sentence after
 * Eq. 2; the container is this library's):
 *   - rank class c = ceil(r / 64); a stored row has 64 c 16-bit elements, the
 *     elements r .. 64c-1 are +0, so reconstruction is exactly rank r;
 *   - a tile = up to 128 tokens of one (layer, K|V, sequence, class); it owns c
 *     consecutive 16 KiB blocks, block j = row-major panel [128 tokens x 64
 *     elements] of elements 64j .. 64j+63; rows past the last token are zero;
 *   - tokens of a (side, sequence, class) fill tiles in arrival order;
 *   - K tiles are listed per class (decode walks classes from wide to narrow),
 *     V tiles per sequence; every V slot links to the score slot of its token.
 */
#ifndef TWKV_H_
#define TWKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TWKV_OK = 0,
  TWKV_ERR_INVALID_ARG = 1,   /* bad pointer, size, id or rank                                  */
  TWKV_ERR_UNSUPPORTED = 2,   /* shape or mode outside the supported set                        */
  TWKV_ERR_CAPACITY = 3,      /* pool, tile tables or per-sequence token limit exhausted        */
  TWKV_ERR_CUDA = 4,          /* a CUDA runtime call failed                                     */
  TWKV_ERR_DEVICE_CHECK = 5,  /* a device-side consistency check failed                         */
  TWKV_ERR_TIMEOUT = 6        /* a bounded device-side wait ran out                             */
} twkv_status;

typedef enum { TWKV_F16 = 0, TWKV_BF16 = 1, TWKV_F32 = 2 } twkv_dtype;

typedef enum {
  TWKV_GATE_FORCED = 0,   /* levels[] is INPUT: the caller gives the ranks                          */
  TWKV_GATE_LOGITS = 1,   /* scores[] is INPUT: gate logits z of Eq. 5; levels[] is OUTPUT          */
  TWKV_GATE_COMPUTE = 2   /* z = x~ W + b is formed from the layer parameters; levels[] is OUTPUT   */
} twkv_gate_mode;

#define TWKV_TILE_TOKENS 128        /* tokens per tile                                               */
#define TWKV_PANEL_ELEMS 64         /* elements per panel row = rank granule                         */
#define TWKV_BLOCK_BYTES 16384      /* one panel: 128 rows x 64 elements x 2 bytes                   */
#define TWKV_PIECE_TOKENS 131072    /* a compress call is processed in pieces of this many tokens    */
#define TWKV_MAX_CLASSES 16
#define TWKV_PREFILL_MAX_QUERIES 16384   /* queries per twkv_prefill_attn call                          */

typedef struct {
  int32_t n_layers;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t head_dim;             /* must be 128                                                       */
  int32_t dtype;                /* twkv_dtype of x~, U^-1, W and q: TWKV_F16 or TWKV_BF16            */
  int32_t out_dtype;            /* twkv_dtype of `out` in twkv_decode_attn (any of the three)        */
  int32_t max_seqs;             /* sequence ids are 0 .. max_seqs-1                                  */
  int32_t max_tokens_per_seq;   /* per layer                                                         */
  float tau;                    /* threshold of Eq. 8 (the paper's example value is 0.1)             */
  float rope_base;              /* RoPE base; pairing (i, i + 64), angle pos * base^(-2i/128)        */
  float sm_scale;               /* softmax scale, usually 1/sqrt(head_dim)                           */
} twkv_config;

typedef struct {
  const void* Uinv_k;   /* [d_kv x d_kv] row-major, dtype; row j = spectral component j (Eq. 3)      */
  const void* Uinv_v;
  const void* W_k;      /* [d_kv x d_kv] row-major, dtype; gate weights of Eq. 5 (may be NULL)       */
  const void* W_v;
  const float* b_k;     /* [d_kv] fp32 gate bias of Eq. 5 (may be NULL = zero)                       */
  const float* b_v;
} twkv_layer_params;

typedef struct {
  uint64_t tokens;                  /* cached tokens in the layer(s)                                 */
  uint64_t bytes_stored;            /* bytes of valid rows, class padding included                   */
  uint64_t bytes_algorithmic;       /* 2 (r_K + r_V) summed over tokens                              */
  uint64_t blocks_used, blocks_free;
  double retain_rate_k;             /* Eq. 4 averaged over tokens                                    */
  double retain_rate_v;
  uint64_t tokens_per_class[2][TWKV_MAX_CLASSES];   /* [K|V][class - 1]                              */
} twkv_stats;

/* Byte offsets (from the start of `pool`) and strides of the cache's tables, for export,
 * inspection and tests.  Per-layer tables are laid out [layer][...]; sides are K = 0, V = 1. */
typedef struct {
  uint64_t pool_bytes, n_blocks, blocks_off;         /* blocks_off: first 16 KiB block               */
  uint64_t status_off;                               /* int32[8]: [0] sticky status, [1] next_block  */
  uint64_t n_tiles_off;                              /* int32 [L][2]                                 */
  uint64_t tile_desc_off;                            /* int32 [L][2][NT][4] = seq, class, n_valid, base block */
  uint64_t tile_aux_off;                             /* int32 [L][2][NT][128]: K position / V score link      */
  uint64_t tile_rank_off;                            /* uint16[L][2][NT][128]                        */
  uint64_t fill_off;                                 /* int32 [L][2*S*NC] tokens per key             */
  uint64_t kclass_count_off, kclass_tiles_off;       /* int32 [L][NC], int32 [L][NC][NT]             */
  uint64_t seq_vcount_off, seq_vtiles_off;           /* int32 [L][S],  int32 [L][S][TPS]             */
  uint64_t seq_tokens_off;                           /* int32 [L][S]                                 */
  uint64_t max_tiles;                                /* NT: tile ids per (layer, side)               */
  uint64_t tiles_per_seq;                            /* TPS                                          */
  uint64_t n_classes;                                /* NC = d_kv / 64                               */
} twkv_layout;

typedef struct twkv_cache twkv_cache;   /* opaque, host memory */

/* Pool size (bytes) that holds `payload_bytes` of packed rows plus worst-case partially
 * filled tiles, all tables and the scratch the two calls use.  Returns 0 if cfg is unsupported. */
size_t twkv_cache_required_bytes(const twkv_config* cfg /*host*/, size_t payload_bytes);

/* Lays the cache out inside pool[0 .. pool_bytes) (256-byte aligned device memory), clears
 * its tables and builds the RoPE tables on `stream`.  *out is host memory owned by the library. */
twkv_status twkv_cache_create(const twkv_config* cfg /*host*/, void* pool, size_t pool_bytes,
                              void* stream, twkv_cache** out /*host*/);
twkv_status twkv_cache_destroy(twkv_cache* cache);
/* Forgets every cached token of every layer (tables cleared, blocks reusable); layer
 * parameters and a pending sticky status are kept / cleared respectively. */
twkv_status twkv_cache_reset(twkv_cache* cache, void* stream);
/* Borrows the layer's matrices (Eq. 3: U^-1; Eq. 5: W, b).  `params` itself is host memory. */
twkv_status twkv_cache_set_layer_params(twkv_cache* cache, int layer, const twkv_layer_params* params /*host*/);

/*
 * Compress step (Eq. 5, 6, 8 for the rank; Eq. 2 for what is stored).
 *   K, V      [n_tok x d_kv] spectral states x~ (pre-RoPE), dtype, row-major
 *   seq_ids   [n_tok] int32, positions [n_tok] int32 (RoPE position of the token)
 *   scores    [n_tok x 2 x d_kv] fp32 gate logits (K row then V row per token); LOGITS mode only, else NULL
 *   levels    [n_tok x 2] uint16 (r_K, r_V): input in FORCED mode (1 <= r <= d_kv), output otherwise
 * Tokens are appended in index order.  A piece of the call (TWKV_PIECE_TOKENS tokens) that does
 * not fit, or that holds an invalid id or rank, is skipped whole and the sticky status is set.
 */
twkv_status twkv_compress(twkv_cache* cache, int layer, const void* K, const void* V,
                          const int32_t* seq_ids, const int32_t* positions, int n_tok,
                          const float* scores, uint16_t* levels, twkv_gate_mode mode, void* stream);

/*
 * Decode attention (Eq. 3, reshape to heads, RoPE on keys, softmax attention) of one query
 * per listed sequence over all tokens cached for that sequence in `layer`.
 *   q        [n_seq x n_q_heads x 128] dtype, already rotated at its own position
 *   seq_ids  [n_seq] int32, distinct
 *   out      [n_seq x n_q_heads x 128] out_dtype; a sequence with no cached token gets zeros
 *   num_splits  V-side splits per sequence; 0 = choose automatically
 */
twkv_status twkv_decode_attn(twkv_cache* cache, int layer, const void* q, const int32_t* seq_ids,
                             int n_seq, void* out, int num_splits, void* stream);

/*
 * Chunked-prefill attention: many causal queries per sequence over the same mixed-rank cache (the paper's
 * long-context evaluation, Sec. 4.2, prefills prompts through the compressed cache; keys and values are the
 * reconstructions of Eq. 3, keys rotated after reconstruction).  Query i attends to the tokens cached for
 * sequence q_seq[i] in `layer` whose position is <= q_pos[i]; the usual order is twkv_compress of a prompt chunk,
 * then this call with the chunk's queries, so that a query also sees its own token.  A query that sees no token
 * gets zeros.
 *   q, out   [n_q x n_q_heads x 128] dtype / out_dtype, device; q already rotated at its own position
 *   q_seq    [n_q] int32, HOST memory: sequence id of every query (any order, repeats allowed)
 *   q_pos    [n_q] int32, HOST memory: RoPE position of every query (>= 0)
 *   n_q      at most TWKV_PREFILL_MAX_QUERIES
 * The queries are served in waves of at most one query per sequence (the k-th query of every sequence together);
 * each wave is one pass of the decode kernels with the causal limit applied to the scores.  The host arrays are
 * read before the call returns.  Errors as for twkv_decode_attn; an id or position out of range returns
 * TWKV_ERR_INVALID_ARG before anything is launched.
 */
twkv_status twkv_prefill_attn(twkv_cache* cache, int layer, const void* q, const int32_t* q_seq /*host*/,
                              const int32_t* q_pos /*host*/, int n_q, void* out, int num_splits, void* stream);

/*
 * Global token eviction with compaction (the paper's combination with token eviction, Sec. 5.2 "Implementation
 * Details" and Table 5: the decomposition is joint across heads, so one token set is kept for all heads).  Of the
 * tokens cached for `seq` in `layer`, exactly those whose position is listed survive, on the K and on the V side.
 *   keep_positions  [n_keep] int32, device, any order; positions nothing is cached at are ignored; n_keep = 0 drops all
 * Container rule: per (side, class) of the sequence the survivors move to the front of the tiles that key owns, in
 * their stored order; vacated rows of the last tile still in use are zeroed; emptied tiles leave the tile lists and
 * their blocks stay unused until twkv_cache_reset; V slots are relinked; later appends continue behind the
 * survivors.  Decode and prefill attention afterwards see the survivors only.
 */
twkv_status twkv_evict(twkv_cache* cache, int layer, int seq, const int32_t* keep_positions, int n_keep, void* stream);

/* Synchronises `stream`, returns the sticky device status and clears it. */
twkv_status twkv_cache_status(twkv_cache* cache, void* stream);
/* Synchronises `stream`; layer = -1 sums all layers.  `out` is host memory. */
twkv_status twkv_cache_stats(twkv_cache* cache, int layer, void* stream, twkv_stats* out /*host*/);
/*
 * Consistency check (a diagnostic of the library; the paper has no counterpart).  A kernel verifies the guard words
 * written behind every region of the pool when the cache was created, and the tables of `layer` (-1 = all): tile
 * descriptors inside their ranges, every stored rank inside its tile's class, every V slot linked to a live K slot of
 * the same sequence, tile lists naming tiles of the right class / sequence.  Synchronises `stream`.  Returns TWKV_OK, or
 * TWKV_ERR_DEVICE_CHECK with the number of violations in *violations (host, may be NULL); the sticky status is set too.
 */
twkv_status twkv_cache_check(twkv_cache* cache, int layer, void* stream, uint64_t* violations /*host*/);
/*
 * Self-test of the bounded device-side wait (diagnostic).  Every tensor-core kernel of the library waits on shared-
 * memory barriers with an attempt limit; a wait that runs out raises its CTA's abort flag, all roles leave their loops
 * and the kernel reports TWKV_ERR_TIMEOUT instead of hanging.  This call launches a one-CTA kernel whose barrier
 * nobody ever completes, with the limit set to `attempts` (the production limit is 2^18, about one second), and synchronises `stream`.
 * Returns TWKV_OK if the wait gave up and raised the flag; the sticky status is then TWKV_ERR_TIMEOUT, as after a
 * production kernel's timeout, until twkv_cache_status reads it.  *elapsed_ns (host, may be NULL) = how long the wait took.
 */
twkv_status twkv_selftest_wait_timeout(twkv_cache* cache, uint32_t attempts, uint64_t* elapsed_ns /*host*/, void* stream);
/* Where the tables live inside the pool (host call, no device work). */
twkv_status twkv_cache_layout(const twkv_cache* cache, twkv_layout* out /*host*/);
/*
 * Soft gating, the differentiable form of the gate the paper trains with, as an inference-time diagnostic:
 *   m = Flip(cumsum(softmax(x~ W + b)))     Eq. 5, Eq. 6 (Flip = index reversal, m_1 = 1, m non-increasing)
 *   x^ = x~ (.) m                           Eq. 7
 *   R = (1/d_kv) sum_i m_i                  the Retain Rate of the soft mask, the R that Eq. 9 penalises
 * for the K side and the V side of n_tok tokens, with the layer's gate parameters (W, b as in TWKV_GATE_COMPUTE).
 * The hard mask of Eq. 8 is this m thresholded at tau.  Nothing is stored in the cache.
 *   K, V          [n_tok x d_kv] spectral states, dtype, device
 *   m_k, m_v      [n_tok x d_kv] fp32 soft masks (each may be NULL)
 *   xh_k, xh_v    [n_tok x d_kv] fp32 gated states (each may be NULL)
 *   retain        [n_tok x 2] fp32 (R_K, R_V) per token (may be NULL)
 */
twkv_status twkv_gate_soft(twkv_cache* cache, int layer, const void* K, const void* V, int n_tok, float* m_k, float* m_v,
                           float* xh_k, float* xh_v, float* retain, void* stream);

/*
 * Gate ranks without any caller-provided scratch (the paper has no counterpart; this is a
 * convenience of the library).  Computes, for n_tok tokens, the (r_K, r_V) of Eq. 5, 6, 8 as twkv_compress
 * does in TWKV_GATE_COMPUTE mode (both evaluate the formulas in fp32; they give the same rank except where a
 * cumulative softmax sum lies within fp32 rounding of tau), but needs no cache and allocates nothing: the
 * fp32 logits are staged in a 4 MiB array that is part of the library image and is resident on
 * every GPU that loads the library, until the process exits.  It is meant for callers that cannot
 * obtain device memory at the point of the call, for instance a scheduler that sizes cache blocks
 * from predicted ranks before a pool exists, or a serving loop whose framework owns all device
 * memory and forbids allocations (which may also synchronise the whole device).
 *   K, V      [n_tok x d_kv] spectral states, `dtype` (TWKV_F16 / TWKV_BF16); W_k, W_v [d_kv x d_kv] `dtype`;
 *   b_k, b_v  [d_kv] fp32 or NULL; levels [n_tok x 2] uint16 OUTPUT; d_kv a multiple of 128, at most 1024
 * Limit: n_tok * 2 * d_kv <= TWKV_STATIC_GATE_MAX_ROWS * 1024 (512 tokens at d_kv = 1024); more returns
 * TWKV_ERR_CAPACITY and launches nothing.  The first call on a device looks the array's address up
 * (a host-side set-up step), so make that first call before any stream capture begins.  All calls on a
 * device share the array: calls that overlap on the GPU (other streams or threads) race; calls queued
 * on one stream are safe.  Nothing has to be cleared between calls.
 */
#define TWKV_STATIC_GATE_MAX_ROWS 1024
twkv_status twkv_gate_ranks_static(const void* K, const void* V, const void* W_k, const void* W_v,
                                   const float* b_k, const float* b_v, int n_tok, int d_kv, int dtype,
                                   float tau, uint16_t* levels, void* stream);

/*
 * Projection to the spectral space (Eq. 1): x~ = x U for the pre-RoPE key and value states, the step
 * right before twkv_compress.  U is the layer's learnable basis (initialised from the PCA eigenvectors,
 * largest eigenvalue first); Eq. 3's U^-1 is its inverse.  The product is accumulated in fp32 from the
 * exact 16-bit inputs and rounded once, to nearest even, into the same 16-bit type: that is the x~ the
 * compress step takes.  Applied to the rows of a model's key / value projection weights instead of to
 * states, the same call folds U into those weights offline (x~ = h (W U)).
 *
 * A projector borrows two things from the caller for its lifetime: nothing of U itself (a transposed
 * copy is made at creation) and `workspace`, device memory of twkv_projector_required_bytes(d_kv) bytes,
 * 256-byte aligned, which holds the copies and a status word.  The library allocates no device memory.
 *   U_k, U_v   [d_kv x d_kv] dtype, row-major, device, 16-byte aligned; row j = input dimension j, column n =
 *              spectral axis n.  Either may be NULL when that side is never projected.
 *   d_kv       multiple of 128, at most 8192
 * twkv_project:
 *   x_k, x_v   [n_tok x d_kv] dtype, row-major, device, 16-byte aligned (input);  NULL skips the side
 *   xt_k, xt_v [n_tok x d_kv] dtype (output); must not overlap the inputs
 * Errors: TWKV_ERR_INVALID_ARG for bad pointers / sizes / a side without its U, TWKV_ERR_CUDA for a failed
 * launch; a device-side wait that ran out shows up as TWKV_ERR_TIMEOUT in twkv_projector_status, which
 * synchronises `stream`, returns the sticky status and clears it.
 */
typedef struct twkv_projector twkv_projector;   /* opaque, host memory */
size_t twkv_projector_required_bytes(int d_kv);
twkv_status twkv_projector_create(int d_kv, twkv_dtype dtype, const void* U_k, const void* U_v, void* workspace,
                                  size_t workspace_bytes, void* stream, twkv_projector** out);
void twkv_projector_destroy(twkv_projector* projector);
twkv_status twkv_project(twkv_projector* projector, const void* x_k, const void* x_v, void* xt_k, void* xt_v,
                         int n_tok, void* stream);
twkv_status twkv_projector_status(twkv_projector* projector, void* stream);

/* Per-kernel device timing.  While enabled, every kernel the library launches for this cache is
 * bracketed by CUDA events on the launching stream (events are host-side resources; no device memory
 * is allocated).  twkv_profile_read synchronises `stream`, adds the elapsed times of the launches
 * recorded since the last read to ms[kind] / launches[kind] (host arrays of TWKV_N_KERNELS entries,
 * overwritten) and forgets them.  At most 8192 launches are kept between reads; later ones are not timed. */
typedef enum {
  TWKV_K_GATE_GEMM = 0, TWKV_K_GATE_RANK = 1, TWKV_K_HIST = 2, TWKV_K_ALLOC = 3, TWKV_K_PACK = 4,
  TWKV_K_PLAN = 5, TWKV_K_KSCORE = 6, TWKV_K_VACC = 7, TWKV_K_MERGE = 8, TWKV_K_OTHER = 9, TWKV_N_KERNELS = 10
} twkv_kernel_kind;
twkv_status twkv_profile_enable(twkv_cache* cache, int enable);
twkv_status twkv_profile_read(twkv_cache* cache, void* stream, double* ms /*host*/, uint64_t* launches /*host*/);
/* Number of kernels this library has launched so far in the process (host counter). */
uint64_t twkv_launch_count(void);
const char* twkv_status_string(twkv_status s);

#ifdef __cplusplus
}
#endif
#endif /* TWKV_H_ */
