"""Shared machinery of the GPU parity tests: run libtwkv through its C ABI, read its tables
back, and compare with the CPU oracle on the same buffers."""
import numpy as np
import torch

import oracle
from oracle.cache_image import CacheImage, TILE, PANEL


def dtype_name(dt):
    return "f16" if dt == torch.float16 else "bf16"


def bits16(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class GpuCache:
    """A cache in a torch-owned pool plus numpy views of its tables."""

    def __init__(self, B, *, n_layers, n_q_heads, n_kv_heads, dtype, out_dtype, max_seqs, max_tokens_per_seq,
                 payload_bytes, tau=0.1, rope_base=500000.0, pool_bytes=None):
        self.B = B
        self.cfg = B.make_config(n_layers=n_layers, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, dtype=dtype,
                                 out_dtype=out_dtype, max_seqs=max_seqs, max_tokens_per_seq=max_tokens_per_seq,
                                 tau=tau, rope_base=rope_base)
        need = B.twkv_cache_required_bytes(self.cfg, payload_bytes) if pool_bytes is None else pool_bytes
        assert need > 0
        self.pool = torch.empty(need, dtype=torch.uint8, device="cuda")
        self.h = B.twkv_cache_create(self.cfg, self.pool)
        self.lay = B.twkv_cache_layout(self.h)
        self.L, self.S = n_layers, max_seqs
        self.d_kv = n_kv_heads * 128

    def close(self):
        self.B.twkv_cache_destroy(self.h)

    def _arr(self, off, count, dt):
        nbytes = count * np.dtype(dt).itemsize
        return self.pool[off:off + nbytes].cpu().numpy().view(dt)

    def tables(self):
        lay = self.lay
        L, S, NT, NC, TPS = self.L, self.S, int(lay.max_tiles), int(lay.n_classes), int(lay.tiles_per_seq)
        t = {}
        t["status"] = self._arr(lay.status_off, 8, np.int32)
        t["n_tiles"] = self._arr(lay.n_tiles_off, L * 2, np.int32).reshape(L, 2)
        t["tile_desc"] = self._arr(lay.tile_desc_off, L * 2 * NT * 4, np.int32).reshape(L, 2, NT, 4)
        t["tile_aux"] = self._arr(lay.tile_aux_off, L * 2 * NT * TILE, np.int32).reshape(L, 2, NT, TILE)
        t["tile_rank"] = self._arr(lay.tile_rank_off, L * 2 * NT * TILE, np.uint16).reshape(L, 2, NT, TILE)
        t["fill"] = self._arr(lay.fill_off, L * 2 * S * NC, np.int32).reshape(L, 2 * S * NC)
        t["kclass_count"] = self._arr(lay.kclass_count_off, L * NC, np.int32).reshape(L, NC)
        t["kclass_tiles"] = self._arr(lay.kclass_tiles_off, L * NC * NT, np.int32).reshape(L, NC, NT)
        t["seq_vcount"] = self._arr(lay.seq_vcount_off, L * S, np.int32).reshape(L, S)
        t["seq_vtiles"] = self._arr(lay.seq_vtiles_off, L * S * TPS, np.int32).reshape(L, S, TPS)
        t["seq_tokens"] = self._arr(lay.seq_tokens_off, L * S, np.int32).reshape(L, S)
        return t

    def blocks(self, n):
        off = int(self.lay.blocks_off)
        return self.pool[off:off + n * 16384].cpu().numpy().view(np.uint16).reshape(n, 8192)


def compare_cache_with_image(gc: GpuCache, img: CacheImage):
    """Bit-exact comparison of every table and every allocated block."""
    t = gc.tables()
    assert t["status"][0] == 0
    assert t["status"][1] == img.next_block
    np.testing.assert_array_equal(t["n_tiles"], img.n_tiles)
    np.testing.assert_array_equal(t["fill"], img.fill)
    np.testing.assert_array_equal(t["seq_tokens"], img.seq_tokens)
    for l in range(img.L):
        for side in range(2):
            n = int(img.n_tiles[l, side])
            np.testing.assert_array_equal(t["tile_desc"][l, side, :n], img.tile_desc[l, side, :n])
            for tid in range(n):
                nv = int(img.tile_desc[l, side, tid, 2])
                np.testing.assert_array_equal(t["tile_aux"][l, side, tid, :nv], img.tile_aux[l, side, tid, :nv])
                np.testing.assert_array_equal(t["tile_rank"][l, side, tid, :nv], img.tile_rank[l, side, tid, :nv])
        for c in range(img.NC):
            want = img.kclass_tiles[l][c]
            assert t["kclass_count"][l, c] == len(want)
            np.testing.assert_array_equal(t["kclass_tiles"][l, c, :len(want)], want)
        for s in range(img.S):
            want = img.seq_vtiles[l][s]
            assert t["seq_vcount"][l, s] == len(want)
            np.testing.assert_array_equal(t["seq_vtiles"][l, s, :len(want)], want)
    if img.next_block:
        np.testing.assert_array_equal(gc.blocks(img.next_block), img.blocks[:img.next_block])


# COMPUTE-mode gate: the library forms z = x~ W + b in fp32 from exact 16-bit products and evaluates Eq. 5, 6, 8 in fp32
# (rows the fused kernel cannot decide from its f16-staged terms are redone from fp32 terms).  With |z| up to a few
# tens, the accumulation error of a logit is below 1e-4 absolute, i.e. below 1e-4 relative on exp(z) and on every
# cumulative sum; decisions the fp64 oracle takes with a relative margin of at least 1e-3 must therefore agree.
GATE_MARGIN_COMPUTE = 1e-3
GATE_MARGIN_LOGITS = 1e-4        # logits given in fp32: only the fp32 softmax and prefix sums differ from fp64


def check_gate_levels(got, z_k, z_v, tau, margin):
    """Per-token ranks of the library against the oracle's gate on the oracle's own logits (Eq. 5, 6, 8).

    Tokens the oracle decides with a relative distance of at least `margin` between every cumulative sum and tau
    must carry the oracle's rank, bit for bit.  For the others several ranks are valid; the rank is non-increasing
    in tau, so the library's rank must lie between the oracle's ranks at tau (1 + margin) and tau (1 - margin).
    Returns the number of (token, side) decisions that fell under the second rule."""
    got = np.asarray(got).astype(np.int64)
    n_loose = 0
    for side, z in enumerate((z_k, z_v)):
        r, m = oracle.gate_rank(z, tau)
        safe = m >= margin
        np.testing.assert_array_equal(got[safe, side], r[safe])
        if not safe.all():
            zz = z[~safe]
            r_lo, _ = oracle.gate_rank(zz, tau * (1.0 + margin))
            r_hi, _ = oracle.gate_rank(zz, tau * (1.0 - margin))
            g = got[~safe, side]
            assert np.all((r_lo <= g) & (g <= r_hi)), (side, g[(g < r_lo) | (g > r_hi)][:8])
            n_loose += int((~safe).sum())
    return n_loose


def oracle_decode(li, ranks, seq_list, layer_tokens=None, rope_base=500000.0):
    """Oracle attention for the listed sequences.  li: LayerInputs (any device); ranks [n, 2] numpy."""
    dn = dtype_name(li.dtype)
    seq_ids = li.seq_ids.cpu().numpy()
    pos = li.positions.cpu().numpy()
    Uk = oracle.widen16(bits16(li.Uinv_k), dn)
    Uv = oracle.widen16(bits16(li.Uinv_v), dn)
    outs = []
    for qi, s in enumerate(seq_list):
        idx = np.nonzero(seq_ids == s)[0]
        xk = oracle.widen16(bits16(li.xt_k[torch.as_tensor(idx, device=li.xt_k.device)]), dn)
        xv = oracle.widen16(bits16(li.xt_v[torch.as_tensor(idx, device=li.xt_v.device)]), dn)
        q = oracle.widen16(bits16(li.q[qi]), dn)
        outs.append(oracle.decode_attn(xk, xv, ranks[idx, 0], ranks[idx, 1], pos[idx], Uk, Uv, q, li.n_kv_heads,
                                       rope_base, li.head_dim ** -0.5))
    return np.stack(outs)


def attn_errors(got, want):
    got = np.asarray(got, dtype=np.float64)
    max_abs = float(np.max(np.abs(got - want)))
    rel_l2 = float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))
    return max_abs, rel_l2
