"""GPU parity of chunked-prefill attention (twkv_prefill_attn through the C ABI) against the CPU oracle.

Every query attends to the cached tokens of its sequence at or before its own position; keys and values are the
rank-r reconstructions of Eq. 3 with keys rotated after reconstruction.  Bars as for decode attention: max-abs 2e-3,
relative L2 1e-3.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_04411_b200 import workloads
from tests.helpers import GpuCache, attn_errors, bits16, dtype_name

pytestmark = pytest.mark.gpu

MAX_ABS, REL_L2 = 2e-3, 1e-3


@pytest.fixture(scope="module")
def B():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding
    return binding


def _oracle_prefill(li, ranks, q, q_seq, q_pos):
    dn = dtype_name(li.dtype)
    seq_ids, pos = li.seq_ids.cpu().numpy(), li.positions.cpu().numpy()
    Uk, Uv = oracle.widen16(bits16(li.Uinv_k), dn), oracle.widen16(bits16(li.Uinv_v), dn)
    xk, xv = oracle.widen16(bits16(li.xt_k), dn), oracle.widen16(bits16(li.xt_v), dn)
    qw = oracle.widen16(bits16(q), dn)
    out = np.zeros(qw.shape)
    for s in np.unique(q_seq):
        rows = np.nonzero(q_seq == s)[0]
        idx = np.nonzero(seq_ids == s)[0]
        out[rows] = oracle.prefill_attn(xk[idx], xv[idx], ranks[idx, 0], ranks[idx, 1], pos[idx], Uk, Uv, qw[rows], q_pos[rows],
                                        li.n_kv_heads, 500000.0, li.head_dim ** -0.5)
    return out


def _case(B, li, ranks, q, q_seq, q_pos, *, calls=None, out_dtype=torch.float32, num_splits=0):
    """Compress the layer (optionally in several calls), run one prefill call, compare with the oracle."""
    n_tok, n_seq = li.xt_k.shape[0], int(li.seq_ids.max()) + 1
    tmax = int(np.bincount(li.seq_ids.numpy(), minlength=n_seq).max())
    gc = GpuCache(B, n_layers=1, n_q_heads=li.n_q_heads, n_kv_heads=li.n_kv_heads, dtype=li.dtype, out_dtype=out_dtype,
                  max_seqs=n_seq, max_tokens_per_seq=tmax, payload_bytes=int((-(-ranks // 64) * 128).sum()))
    dev = [t.cuda().contiguous() for t in (li.Uinv_k, li.Uinv_v, li.xt_k, li.xt_v, li.seq_ids, li.positions)]
    B.twkv_cache_set_layer_params(gc.h, 0, dev[0], dev[1])
    lv = torch.from_numpy(ranks.astype(np.int16)).cuda().contiguous()
    for lo, hi in (calls or [(0, n_tok)]):
        B.twkv_compress(gc.h, 0, dev[2][lo:hi], dev[3][lo:hi], dev[4][lo:hi], dev[5][lo:hi], None, lv[lo:hi], B.TWKV_GATE_FORCED)
    out = torch.full((len(q_seq), li.n_q_heads, 128), float("nan"), dtype=out_dtype, device="cuda")
    B.twkv_prefill_attn(gc.h, 0, q.cuda().contiguous(), q_seq, q_pos, out, num_splits)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    got = out.float().cpu().numpy()
    assert np.all(np.isfinite(got))
    want = _oracle_prefill(li, ranks, q, np.asarray(q_seq), np.asarray(q_pos))
    gc.close()
    return attn_errors(got, want), got, want


@pytest.mark.parametrize("chunk", [1, 127, 128, 129])
def test_prefill_chunk_sizes(B, chunk):
    # one sequence of 300 cached tokens (any rank, K and V independent), the last `chunk` tokens are the prompt chunk:
    # their queries attend causally, the chunk straddles tile boundaries of several rank classes
    li = workloads.build_layer(500 + chunk, n_seq=1, ctx=300, n_q_heads=32, mode="forced", rank_recipe="any", outlier="pct:1")
    ranks = li.ranks.numpy().astype(np.int64)
    g = torch.Generator().manual_seed(chunk)
    q = torch.randn(chunk, 32, 128, generator=g).to(torch.float16)
    q_pos = np.arange(300 - chunk, 300)
    (max_abs, rel_l2), _, _ = _case(B, li, ranks, q, np.zeros(chunk, np.int64), q_pos)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_prefill_three_sequences_uneven_chunks_bf16(B):
    # bf16, GQA 8, three sequences with chunks of 5, 1 and 40 queries listed interleaved; shuffled cache positions, a
    # query before every cached token (zeros), and queries that repeat a position
    li = workloads.build_layer(611, n_seq=3, ctx=260, n_q_heads=64, dtype=torch.bfloat16, mode="forced", outlier="t3pct:1",
                               level_probs=(0.1, 0.2, 0.4, 0.3), shuffle_positions=True)
    li.positions = li.positions + 3                                         # nothing is cached at positions 0..2
    ranks = li.ranks.numpy().astype(np.int64)
    rng = np.random.default_rng(3)
    q_seq = np.array([0] * 5 + [1] + [2] * 40)
    q_pos = np.concatenate([[1, 3, 100, 100, 262], [50], rng.integers(3, 263, 40)])
    perm = rng.permutation(len(q_seq))
    q_seq, q_pos = q_seq[perm], q_pos[perm]
    g = torch.Generator().manual_seed(7)
    q = torch.randn(len(q_seq), 64, 128, generator=g).to(torch.bfloat16)
    (max_abs, rel_l2), got, want = _case(B, li, ranks, q, q_seq, q_pos)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    assert not got[(q_seq == 0) & (q_pos == 1)].any()                       # the query at position 1 sees no token


def test_prefill_after_chunked_compress_equals_decode_for_the_last_query(B):
    # prompt fed in two chunks; the last query of the second chunk sees everything, so it must agree with decode
    li = workloads.build_layer(701, n_seq=2, ctx=200, n_q_heads=32, mode="forced", outlier="pct:1")
    order = torch.cat([torch.arange(0, 120), torch.arange(200, 320), torch.arange(120, 200), torch.arange(320, 400)])
    for name in ["xt_k", "xt_v", "seq_ids", "positions", "ranks"]:
        setattr(li, name, getattr(li, name)[order].contiguous())
    ranks = li.ranks.numpy().astype(np.int64)
    q_seq = np.array([0] * 80 + [1] * 80)
    q_pos = np.concatenate([np.arange(120, 200), np.arange(120, 200)])
    g = torch.Generator().manual_seed(9)
    q = torch.randn(160, 32, 128, generator=g).to(torch.float16)
    (max_abs, rel_l2), got, _ = _case(B, li, ranks, q, q_seq, q_pos, calls=[(0, 240), (240, 400)])
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    # the same cache, decode with the two last queries
    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32, max_seqs=2,
                  max_tokens_per_seq=200, payload_bytes=int((-(-ranks // 64) * 128).sum()))
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k.cuda(), li.Uinv_v.cuda())
    B.twkv_compress(gc.h, 0, li.xt_k.cuda(), li.xt_v.cuda(), li.seq_ids.cuda(), li.positions.cuda(), None,
                    torch.from_numpy(ranks.astype(np.int16)).cuda(), B.TWKV_GATE_FORCED)
    out = torch.empty(2, 32, 128, device="cuda")
    B.twkv_decode_attn(gc.h, 0, q[[79, 159]].cuda().contiguous(), torch.tensor([0, 1], dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    np.testing.assert_allclose(out.cpu().numpy(), got[[79, 159]], rtol=0, atol=1e-6)
    # argument errors are returned before anything runs
    for bad_seq, bad_pos in (([2], [0]), ([0], [-1])):
        with pytest.raises(B.TwkvError) as err:
            B.twkv_prefill_attn(gc.h, 0, q[:1].cuda().contiguous(), bad_seq, bad_pos, out[:1])
        assert err.value.code == B.TWKV_ERR_INVALID_ARG
    gc.close()
