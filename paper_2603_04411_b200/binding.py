"""Thin ctypes binding of libtwkv's C ABI (argument marshalling only).

Every function has the name and the meaning of its C counterpart in
include/twkv.h; tensors are torch CUDA tensors whose data pointers are handed
through unchanged.  There is no fallback: if libtwkv.so is missing or cannot be
loaded, importing this module raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtwkv.so")

TWKV_OK, TWKV_ERR_INVALID_ARG, TWKV_ERR_UNSUPPORTED, TWKV_ERR_CAPACITY = 0, 1, 2, 3
TWKV_ERR_CUDA, TWKV_ERR_DEVICE_CHECK, TWKV_ERR_TIMEOUT = 4, 5, 6
TWKV_F16, TWKV_BF16, TWKV_F32 = 0, 1, 2
TWKV_GATE_FORCED, TWKV_GATE_LOGITS, TWKV_GATE_COMPUTE = 0, 1, 2
TILE_TOKENS, PANEL_ELEMS, BLOCK_BYTES, PIECE_TOKENS, MAX_CLASSES = 128, 64, 16384, 131072, 16
PREFILL_MAX_QUERIES = 16384

EXPORTS = ["twkv_cache_required_bytes", "twkv_cache_create", "twkv_cache_destroy", "twkv_cache_reset",
           "twkv_cache_set_layer_params", "twkv_compress", "twkv_decode_attn", "twkv_prefill_attn", "twkv_evict", "twkv_cache_check", "twkv_selftest_wait_timeout", "twkv_cache_status",
           "twkv_cache_stats", "twkv_cache_layout", "twkv_launch_count", "twkv_status_string",
           "twkv_profile_enable", "twkv_profile_read", "twkv_gate_ranks_static", "twkv_gate_soft",
           "twkv_projector_required_bytes", "twkv_projector_create", "twkv_projector_destroy", "twkv_project",
           "twkv_projector_status"]
STATIC_GATE_MAX_ROWS = 1024
KERNEL_KINDS = ["gate_gemm", "gate_rank", "hist", "alloc", "pack", "plan", "kscore", "vacc", "merge", "other"]


class twkv_config(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
                ("max_seqs", ctypes.c_int32), ("max_tokens_per_seq", ctypes.c_int32),
                ("tau", ctypes.c_float), ("rope_base", ctypes.c_float), ("sm_scale", ctypes.c_float)]


class twkv_layer_params(ctypes.Structure):
    _fields_ = [("Uinv_k", ctypes.c_void_p), ("Uinv_v", ctypes.c_void_p), ("W_k", ctypes.c_void_p),
                ("W_v", ctypes.c_void_p), ("b_k", ctypes.c_void_p), ("b_v", ctypes.c_void_p)]


class twkv_stats(ctypes.Structure):
    _fields_ = [("tokens", ctypes.c_uint64), ("bytes_stored", ctypes.c_uint64), ("bytes_algorithmic", ctypes.c_uint64),
                ("blocks_used", ctypes.c_uint64), ("blocks_free", ctypes.c_uint64),
                ("retain_rate_k", ctypes.c_double), ("retain_rate_v", ctypes.c_double),
                ("tokens_per_class", (ctypes.c_uint64 * MAX_CLASSES) * 2)]


class twkv_layout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in
                ["pool_bytes", "n_blocks", "blocks_off", "status_off", "n_tiles_off", "tile_desc_off", "tile_aux_off",
                 "tile_rank_off", "fill_off", "kclass_count_off", "kclass_tiles_off", "seq_vcount_off",
                 "seq_vtiles_off", "seq_tokens_off", "max_tiles", "tiles_per_seq", "n_classes"]]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_04411_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.twkv_cache_required_bytes.argtypes = [ctypes.POINTER(twkv_config), sz]
    L.twkv_cache_required_bytes.restype = sz
    L.twkv_cache_create.argtypes = [ctypes.POINTER(twkv_config), vp, sz, vp, ctypes.POINTER(vp)]
    L.twkv_cache_destroy.argtypes = [vp]
    L.twkv_cache_reset.argtypes = [vp, vp]
    L.twkv_cache_set_layer_params.argtypes = [vp, i32, ctypes.POINTER(twkv_layer_params)]
    L.twkv_compress.argtypes = [vp, i32, vp, vp, vp, vp, i32, vp, vp, i32, vp]
    L.twkv_decode_attn.argtypes = [vp, i32, vp, vp, i32, vp, i32, vp]
    L.twkv_prefill_attn.argtypes = [vp, i32, vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32), i32, vp, i32, vp]
    L.twkv_cache_check.argtypes = [vp, i32, vp, ctypes.POINTER(ctypes.c_uint64)]
    L.twkv_cache_check.restype = i32
    L.twkv_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint64), vp]
    L.twkv_selftest_wait_timeout.restype = i32
    L.twkv_evict.argtypes = [vp, i32, i32, vp, i32, vp]
    L.twkv_evict.restype = i32
    L.twkv_gate_soft.argtypes = [vp, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.twkv_gate_soft.restype = i32
    L.twkv_cache_status.argtypes = [vp, vp]
    L.twkv_cache_stats.argtypes = [vp, i32, vp, ctypes.POINTER(twkv_stats)]
    L.twkv_cache_layout.argtypes = [vp, ctypes.POINTER(twkv_layout)]
    L.twkv_profile_enable.argtypes = [vp, i32]
    L.twkv_profile_read.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_uint64)]
    L.twkv_gate_ranks_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, ctypes.c_float, vp, vp]
    L.twkv_gate_ranks_static.restype = i32
    L.twkv_projector_required_bytes.argtypes = [i32]
    L.twkv_projector_required_bytes.restype = sz
    L.twkv_projector_create.argtypes = [i32, i32, vp, vp, vp, sz, vp, ctypes.POINTER(vp)]
    L.twkv_projector_create.restype = i32
    L.twkv_projector_destroy.argtypes = [vp]
    L.twkv_projector_destroy.restype = None
    L.twkv_project.argtypes = [vp, vp, vp, vp, vp, i32, vp]
    L.twkv_project.restype = i32
    L.twkv_projector_status.argtypes = [vp, vp]
    L.twkv_projector_status.restype = i32
    L.twkv_launch_count.argtypes = []
    L.twkv_launch_count.restype = ctypes.c_uint64
    L.twkv_status_string.argtypes = [i32]
    L.twkv_status_string.restype = ctypes.c_char_p
    for name in ["twkv_cache_create", "twkv_cache_destroy", "twkv_cache_reset", "twkv_cache_set_layer_params",
                 "twkv_compress", "twkv_decode_attn", "twkv_prefill_attn", "twkv_cache_status", "twkv_cache_stats", "twkv_cache_layout",
                 "twkv_profile_enable", "twkv_profile_read"]:
        getattr(L, name).restype = i32
    return L


lib = _load()


class TwkvError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib.twkv_status_string(code).decode()} ({code})")


def _check(code, where):
    if code != TWKV_OK:
        raise TwkvError(code, where)


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "libtwkv takes contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def dtype_code(dt) -> int:
    return {torch.float16: TWKV_F16, torch.bfloat16: TWKV_BF16, torch.float32: TWKV_F32}[dt]


def make_config(*, n_layers, n_q_heads, n_kv_heads, head_dim=128, dtype=torch.float16, out_dtype=None,
                max_seqs, max_tokens_per_seq, tau=0.1, rope_base=500000.0, sm_scale=None) -> twkv_config:
    return twkv_config(n_layers, n_q_heads, n_kv_heads, head_dim, dtype_code(dtype),
                       dtype_code(out_dtype if out_dtype is not None else dtype), max_seqs, max_tokens_per_seq,
                       tau, rope_base, sm_scale if sm_scale is not None else head_dim ** -0.5)


def twkv_cache_required_bytes(cfg: twkv_config, payload_bytes: int) -> int:
    return int(lib.twkv_cache_required_bytes(ctypes.byref(cfg), payload_bytes))


def twkv_cache_create(cfg: twkv_config, pool: torch.Tensor, stream=None):
    """pool: 1-D uint8 CUDA tensor owned by the caller (kept alive by the caller)."""
    h = ctypes.c_void_p()
    _check(lib.twkv_cache_create(ctypes.byref(cfg), _ptr(pool), pool.numel() * pool.element_size(), _stream(stream),
                                 ctypes.byref(h)), "twkv_cache_create")
    return h


def twkv_cache_destroy(cache):
    _check(lib.twkv_cache_destroy(cache), "twkv_cache_destroy")
    _borrowed.pop(cache.value, None)


def twkv_cache_reset(cache, stream=None):
    _check(lib.twkv_cache_reset(cache, _stream(stream)), "twkv_cache_reset")


# The library borrows a layer's parameter tensors until the cache is destroyed or the parameters are replaced.  The
# binding keeps a reference to them for that long, so that a caller who passes temporaries (x.cuda()) does not leave the
# cache with pointers into memory the allocator has taken back.
_borrowed = {}


def twkv_cache_set_layer_params(cache, layer, Uinv_k, Uinv_v, W_k=None, W_v=None, b_k=None, b_v=None):
    p = twkv_layer_params(_ptr(Uinv_k), _ptr(Uinv_v), _ptr(W_k), _ptr(W_v), _ptr(b_k), _ptr(b_v))
    _check(lib.twkv_cache_set_layer_params(cache, layer, ctypes.byref(p)), "twkv_cache_set_layer_params")
    _borrowed.setdefault(cache.value, {})[layer] = (Uinv_k, Uinv_v, W_k, W_v, b_k, b_v)


def twkv_compress(cache, layer, K, V, seq_ids, positions, scores, levels, mode, stream=None, n_tok=None):
    n = K.shape[0] if n_tok is None else n_tok
    _check(lib.twkv_compress(cache, layer, _ptr(K), _ptr(V), _ptr(seq_ids), _ptr(positions), n, _ptr(scores),
                             _ptr(levels), mode, _stream(stream)), "twkv_compress")


def twkv_decode_attn(cache, layer, q, seq_ids, out, num_splits=0, stream=None):
    _check(lib.twkv_decode_attn(cache, layer, _ptr(q), _ptr(seq_ids), seq_ids.numel(), _ptr(out), num_splits,
                                _stream(stream)), "twkv_decode_attn")


def twkv_prefill_attn(cache, layer, q, q_seq, q_pos, out, num_splits=0, stream=None):
    """Causal attention of a chunk of queries over the cache.  q / out: [n_q, Hq, 128] CUDA tensors; q_seq / q_pos:
    the queries' sequence ids and positions as HOST integers (lists, numpy arrays or CPU tensors)."""
    seq = [int(x) for x in q_seq]
    pos = [int(x) for x in q_pos]
    n = len(seq)
    assert len(pos) == n and q.shape[0] == n
    arr = ctypes.c_int32 * max(n, 1)
    _check(lib.twkv_prefill_attn(cache, layer, _ptr(q), arr(*seq), arr(*pos), n, _ptr(out), num_splits, _stream(stream)),
           "twkv_prefill_attn")


def twkv_cache_check(cache, layer=-1, stream=None):
    """-> (status code, number of violations): guard words and table invariants, checked by a kernel."""
    bad = ctypes.c_uint64(0)
    code = int(lib.twkv_cache_check(cache, layer, _stream(stream), ctypes.byref(bad)))
    return code, int(bad.value)


def twkv_selftest_wait_timeout(cache, attempts, stream=None):
    """-> (status code, elapsed ns) of a bounded wait that nobody ends; leaves TWKV_ERR_TIMEOUT as the sticky status."""
    ns = ctypes.c_uint64(0)
    code = int(lib.twkv_selftest_wait_timeout(cache, attempts, ctypes.byref(ns), _stream(stream)))
    return code, int(ns.value)


def twkv_evict(cache, layer, seq, keep_positions, stream=None):
    """Keeps, of sequence `seq` in `layer`, only the tokens at the listed positions (int32 CUDA tensor) and compacts them."""
    _check(lib.twkv_evict(cache, layer, seq, _ptr(keep_positions), keep_positions.numel(), _stream(stream)), "twkv_evict")


def twkv_gate_soft(cache, layer, K, V, m_k=None, m_v=None, xh_k=None, xh_v=None, retain=None, stream=None, n_tok=None):
    """Soft mask m (Eq. 6), gated states x~ (.) m (Eq. 7) and the soft mask's Retain Rate per token, fp32 outputs."""
    n = K.shape[0] if n_tok is None else n_tok
    _check(lib.twkv_gate_soft(cache, layer, _ptr(K), _ptr(V), n, _ptr(m_k), _ptr(m_v), _ptr(xh_k), _ptr(xh_v), _ptr(retain),
                              _stream(stream)), "twkv_gate_soft")


def twkv_cache_status(cache, stream=None) -> int:
    return int(lib.twkv_cache_status(cache, _stream(stream)))


def twkv_cache_stats(cache, layer=-1, stream=None) -> twkv_stats:
    st = twkv_stats()
    _check(lib.twkv_cache_stats(cache, layer, _stream(stream), ctypes.byref(st)), "twkv_cache_stats")
    return st


def twkv_cache_layout(cache) -> twkv_layout:
    lay = twkv_layout()
    _check(lib.twkv_cache_layout(cache, ctypes.byref(lay)), "twkv_cache_layout")
    return lay


def twkv_profile_enable(cache, enable: bool):
    _check(lib.twkv_profile_enable(cache, 1 if enable else 0), "twkv_profile_enable")


def twkv_profile_read(cache, stream=None):
    """-> {kernel name: (total ms, launches)} since the last read."""
    n = len(KERNEL_KINDS)
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_uint64 * n)()
    _check(lib.twkv_profile_read(cache, _stream(stream), ms, cnt), "twkv_profile_read")
    return {k: (ms[i], int(cnt[i])) for i, k in enumerate(KERNEL_KINDS)}


def twkv_gate_ranks_static(K, V, W_k, W_v, b_k, b_v, levels, tau=0.1, stream=None, n_tok=None):
    """Gate ranks for a few tokens with the logits staged in the library's own fixed 4 MiB device
    array: no cache, no pool, no allocation.  For callers that cannot get device memory when they
    need the ranks (see include/twkv.h).  At most 512 tokens at d_kv = 1024; calls that overlap on
    the GPU share that array and race, calls on one stream do not."""
    n = K.shape[0] if n_tok is None else n_tok
    _check(lib.twkv_gate_ranks_static(_ptr(K), _ptr(V), _ptr(W_k), _ptr(W_v), _ptr(b_k), _ptr(b_v), n, K.shape[1],
                                      dtype_code(K.dtype), tau, _ptr(levels), _stream(stream)), "twkv_gate_ranks_static")


def twkv_projector_required_bytes(d_kv: int) -> int:
    return int(lib.twkv_projector_required_bytes(d_kv))


def twkv_projector_create(U_k, U_v, workspace: torch.Tensor, stream=None):
    """U_k / U_v: [d_kv, d_kv] fp16 or bf16 CUDA tensors (either may be None); workspace: 1-D uint8 CUDA tensor of
    twkv_projector_required_bytes(d_kv) bytes owned by the caller (kept alive by the caller)."""
    U = U_k if U_k is not None else U_v
    h = ctypes.c_void_p()
    _check(lib.twkv_projector_create(U.shape[0], dtype_code(U.dtype), _ptr(U_k), _ptr(U_v), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream), ctypes.byref(h)),
           "twkv_projector_create")
    return h


def twkv_projector_destroy(projector):
    lib.twkv_projector_destroy(projector)


def twkv_project(projector, x_k, x_v, xt_k, xt_v, stream=None, n_tok=None):
    """Eq. 1 on the device: xt = x U for the pre-RoPE key and / or value states ([n_tok, d_kv], 16-bit)."""
    x = x_k if x_k is not None else x_v
    n = (x.shape[0] if x is not None else 0) if n_tok is None else n_tok
    _check(lib.twkv_project(projector, _ptr(x_k), _ptr(x_v), _ptr(xt_k), _ptr(xt_v), n, _stream(stream)), "twkv_project")


def twkv_projector_status(projector, stream=None) -> int:
    return int(lib.twkv_projector_status(projector, _stream(stream)))


def twkv_launch_count() -> int:
    return int(lib.twkv_launch_count())


def twkv_status_string(code: int) -> str:
    return lib.twkv_status_string(code).decode()
