"""fp64 CPU oracle (ctypes front end of oracle/twkv_oracle.c).

TEST INFRASTRUCTURE ONLY.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the product library never does, and
this package never imports the product library.

All floating point goes through float64.  16-bit inputs (fp16 / bf16 bit
patterns, exactly as the GPU receives them) are widened with `widen16`.

  project(x, U)                    Eq. 1   x~ = x U
  narrow16(a, dtype)               float64 -> the 16-bit storage type, round to nearest even
  gate_logits(xt, W, b)            Eq. 5   z = x~ W + b
  gate_rank(z, tau)                Eq. 5, 6, 8   -> (r, margin[, soft mask])
  truncate(xt, r)                  Eq. 2   x^ = x~ (.) m_hard
  reconstruct(xt, r, Uinv)         Eq. 3   xbar = x^[I] Uinv[I, :]
  rope(k, pos, n_heads, d_h, base) RoPE on reconstructed keys (after Eq. 3)
  decode_attn(...)                 Eq. 3 + reshape + RoPE + softmax attention, one sequence
  prefill_attn(...)                the same for many causal queries of one sequence (a prompt chunk)
  soft_gate(xt, z)                 Eq. 6, Eq. 7, Eq. 9's R: soft mask m, x~ (.) m, mean of m per token
  retain_rate(r, d)                Eq. 4   mean of r / d_kv
"""
import ctypes
import os

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        path = _build.build()
        L = ctypes.CDLL(path)
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_project.argtypes = [dp, dp, ctypes.c_int64, ctypes.c_int, dp]
        L.oracle_project.restype = None
        L.oracle_gate_logits.argtypes = [dp, dp, dp, ctypes.c_int64, ctypes.c_int, dp]
        L.oracle_gate_logits.restype = None
        L.oracle_gate_rank.argtypes = [dp, ctypes.c_int64, ctypes.c_int, ctypes.c_double, ip, dp, dp]
        L.oracle_gate_rank.restype = None
        L.oracle_reconstruct.argtypes = [dp, ip, dp, ctypes.c_int64, ctypes.c_int, dp]
        L.oracle_reconstruct.restype = None
        L.oracle_rope.argtypes = [dp, ip, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_double]
        L.oracle_rope.restype = None
        L.oracle_decode_attn.argtypes = [dp, dp, ip, ip, ip, ctypes.c_int64, dp, dp, dp,
                                         ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_double, ctypes.c_double, dp]
        L.oracle_decode_attn.restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _i(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def widen16(bits, dtype: str) -> np.ndarray:
    """uint16 bit patterns of fp16 ('f16') or bf16 ('bf16') values -> float64, exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == "f16":
        return bits.view(np.float16).astype(np.float64)
    if dtype == "bf16":
        return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    raise ValueError(dtype)


def narrow16(a, dtype: str) -> np.ndarray:
    """float64 -> uint16 bit patterns of fp16 ('f16') or bf16 ('bf16'), round to nearest even.

    The states handed to the compress step are 16-bit; this is the one rounding between Eq. 1 and Eq. 2.
    Both conversions go through a single rounding of the float64 value (no intermediate float32 rounding
    that could double-round): numpy's float64 -> float16 cast for fp16, integer arithmetic on the float64
    bit pattern for bf16.  Overflow gives infinity, as IEEE round-to-nearest does.
    """
    a = np.ascontiguousarray(a, dtype=np.float64)
    if dtype == "f16":
        with np.errstate(over="ignore"):
            return a.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        # bf16 has float32's exponent range and 8 significand bits; values are assumed normal in float32
        # (|a| >= 2^-126 or a == 0), which holds for every state the tests and workloads produce.
        m, e = np.frexp(a)                                  # a = m 2^e, 0.5 <= |m| < 1
        q = np.rint(np.ldexp(m, 8))                         # 8 significant bits, ties to even (rint)
        v = np.ldexp(q, e - 8)                              # exactly representable in bf16 (or overflows below)
        with np.errstate(over="ignore"):
            f = v.astype(np.float32)                        # exact: v has 8 significant bits
        return (f.view(np.uint32) >> 16).astype(np.uint16)
    raise ValueError(dtype)


def project(x, U) -> np.ndarray:
    """Eq. 1: x~ = x U.  x [n, d] pre-RoPE states, U [d, d]."""
    x, px = _d(x)
    U, pU = _d(U)
    n, d = x.shape
    assert U.shape == (d, d)
    xt = np.empty((n, d), dtype=np.float64)
    lib().oracle_project(px, pU, n, d, xt.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    return xt


def gate_logits(xt, W, b=None) -> np.ndarray:
    """Eq. 5, argument of the softmax: z = x~ W + b.  xt [n, d], W [d, d], b [d]."""
    xt, pxt = _d(xt)
    W, pW = _d(W)
    n, d = xt.shape
    assert W.shape == (d, d)
    z = np.empty((n, d), dtype=np.float64)
    if b is None:
        pb = None
    else:
        b, pb = _d(b)
    lib().oracle_gate_logits(pxt, pW, pb, n, d, z.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    return z


def gate_rank(z, tau: float, want_soft: bool = False):
    """Eq. 5, 6, 8 -> retained rank r [n] (int32), margin [n], optional soft mask [n, d]."""
    z, pz = _d(z)
    n, d = z.shape
    r = np.empty(n, dtype=np.int32)
    margin = np.empty(n, dtype=np.float64)
    m = np.empty((n, d), dtype=np.float64) if want_soft else None
    lib().oracle_gate_rank(pz, n, d, float(tau),
                           r.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                           margin.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                           m.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if want_soft else None)
    return (r, margin, m) if want_soft else (r, margin)


def truncate(xt, r) -> np.ndarray:
    """Eq. 2: x^ = x~ (.) m_hard, m_hard = r ones followed by zeros."""
    xt = np.asarray(xt)
    d = xt.shape[-1]
    mask = np.arange(d)[None, :] < np.asarray(r)[:, None]
    return np.where(mask, xt, np.zeros((), dtype=xt.dtype))


def reconstruct(xt, r, Uinv) -> np.ndarray:
    """Eq. 3: xbar = x^[I] Uinv[I, :] with I = {0..r-1} per token."""
    xt, pxt = _d(xt)
    Uinv, pU = _d(Uinv)
    r, pr = _i(r)
    n, d = xt.shape
    out = np.empty((n, d), dtype=np.float64)
    lib().oracle_reconstruct(pxt, pr, pU, n, d, out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    return out


def rope(k, pos, n_heads: int, d_h: int, base: float) -> np.ndarray:
    """RoPE (rotate-half pairing) on keys k [n, n_heads*d_h]; returns a rotated copy."""
    k = np.array(k, dtype=np.float64, order="C", copy=True)
    pos, pp = _i(pos)
    n = k.shape[0]
    lib().oracle_rope(k.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), pp, n, n_heads, d_h, float(base))
    return k


def decode_attn(xk, xv, rk, rv, pos, Uinv_k, Uinv_v, q, n_kv_heads: int,
                rope_base: float, sm_scale: float) -> np.ndarray:
    """One decode step for one sequence.  xk/xv [T, d_kv]; q [Hq, d_h] -> out [Hq, d_h]."""
    xk, pxk = _d(xk)
    xv, pxv = _d(xv)
    rk, prk = _i(rk)
    rv, prv = _i(rv)
    pos, ppos = _i(pos)
    Uinv_k, pUk = _d(Uinv_k)
    Uinv_v, pUv = _d(Uinv_v)
    q, pq = _d(q)
    T, d = xk.shape
    Hq, d_h = q.shape
    assert d == n_kv_heads * d_h and Hq % n_kv_heads == 0
    out = np.empty((Hq, d_h), dtype=np.float64)
    rc = lib().oracle_decode_attn(pxk, pxv, prk, prv, ppos, T, pUk, pUv, pq, Hq, n_kv_heads, d_h,
                                  float(rope_base), float(sm_scale),
                                  out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc != 0:
        raise MemoryError("oracle_decode_attn")
    return out


def prefill_attn(xk, xv, rk, rv, pos, Uinv_k, Uinv_v, q, q_pos, n_kv_heads: int,
                 rope_base: float, sm_scale: float) -> np.ndarray:
    """Attention of a chunk of causal queries over one sequence's cached tokens.

    The paper's long-context evaluation (Sec. 4.2) prefills prompts through the same compressed cache: every query
    sees the reconstructed keys and values of Eq. 3 (keys rotated after reconstruction) of the tokens at or before
    its own position.  This is that definition written out: query i attends to the cached tokens t with
    pos[t] <= q_pos[i], each such set handed to decode_attn unchanged; a query that sees no token gets zeros.
    xk/xv [T, d_kv], q [n_q, Hq, d_h], q_pos [n_q] -> out [n_q, Hq, d_h]."""
    q = np.asarray(q, dtype=np.float64)
    pos = np.asarray(pos)
    out = np.zeros(q.shape, dtype=np.float64)
    for i in range(q.shape[0]):
        vis = np.nonzero(pos <= q_pos[i])[0]
        if len(vis):
            out[i] = decode_attn(np.asarray(xk)[vis], np.asarray(xv)[vis], np.asarray(rk)[vis], np.asarray(rv)[vis], pos[vis],
                                 Uinv_k, Uinv_v, q[i], n_kv_heads, rope_base, sm_scale)
    return out


def soft_gate(xt, z):
    """Soft gating of Eq. 6 and Eq. 7, and the per-token Retain Rate of the soft mask that Eq. 9 penalises.

    m = Flip(cumsum(softmax(z))) (Eq. 6, the literal index reversal m_i = c_{d+1-i}); x^ = x~ (.) m (Eq. 7);
    R = (1/d) sum_i m_i, Eq. 4 applied to the soft mask.  xt, z [n, d] -> (m [n, d], x^ [n, d], R [n])."""
    xt = np.asarray(xt, dtype=np.float64)
    _, _, m = gate_rank(z, 0.5, want_soft=True)
    return m, xt * m, m.mean(axis=1)


def retain_rate(r, d: int) -> float:
    """Eq. 4 averaged over the given tokens: mean(r) / d_kv."""
    return float(np.mean(np.asarray(r, dtype=np.float64)) / d)
