"""GPU parity: libtwkv (through its C ABI) against the fp64 CPU oracle on the same seeded inputs.

Bars: ranks, tables and packed bytes bit-exact; attention output within max-abs 2e-3 and
relative L2 1e-3 of the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle.cache_image import CacheImage
from paper_2603_04411_b200 import workloads
from tests.helpers import GATE_MARGIN_LOGITS, GpuCache, attn_errors, bits16, compare_cache_with_image, oracle_decode

pytestmark = pytest.mark.gpu

MAX_ABS, REL_L2 = 2e-3, 1e-3


@pytest.fixture(scope="module")
def B():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding
    return binding


def to_cuda(li):
    for name in ["Uinv_k", "Uinv_v", "xt_k", "xt_v", "seq_ids", "positions", "q", "logits"]:
        t = getattr(li, name)
        if t is not None:
            setattr(li, name, t.cuda().contiguous())
    return li


def levels_tensor(ranks_np):
    return torch.from_numpy(np.ascontiguousarray(ranks_np.astype(np.int16))).cuda().contiguous()


def settle_logits(logits, tau, min_margin):
    """Margin protocol: rows whose cumulative softmax comes within min_margin (relative) of tau are
    replaced by rows that jump across tau at one index, so the integer rank cannot depend on rounding."""
    n, _, d = logits.shape
    z = logits.reshape(n * 2, d).double().numpy()
    r, margin = oracle.gate_rank(z, tau)
    bad = np.nonzero(margin < min_margin)[0]
    for i in bad:
        logits.reshape(n * 2, d)[i] = workloads.safe_logit_row(d, int(r[i]))
    if len(bad):
        z = logits.reshape(n * 2, d).double().numpy()
        r, margin = oracle.gate_rank(z, tau)
        assert margin.min() >= min_margin
    return r.reshape(n, 2), len(bad)


def run_case(B, li, ranks_np, *, mode, out_dtype=torch.float32, calls=None, n_layers=1, layer=0, num_splits=0,
             max_tokens_per_seq=None, check_image=True, decode_seqs=None):
    """Compress (optionally in several calls), compare the cache image, decode, compare with the oracle."""
    n_tok = li.xt_k.shape[0]
    n_seq = li.q.shape[0]
    seq_np = li.seq_ids.cpu().numpy()
    pos_np = li.positions.cpu().numpy()
    tmax = max_tokens_per_seq or int(np.bincount(seq_np, minlength=n_seq).max())
    payload = int((-(-ranks_np // 64) * 128).sum())
    gc = GpuCache(B, n_layers=n_layers, n_q_heads=li.n_q_heads, n_kv_heads=li.n_kv_heads, dtype=li.dtype,
                  out_dtype=out_dtype, max_seqs=n_seq, max_tokens_per_seq=tmax, payload_bytes=payload)
    B.twkv_cache_set_layer_params(gc.h, layer, li.Uinv_k, li.Uinv_v)
    levels = levels_tensor(ranks_np) if mode == B.TWKV_GATE_FORCED else torch.zeros(n_tok, 2, dtype=torch.int16, device="cuda")
    img = CacheImage(n_layers, li.d_kv, n_seq, tmax, int(gc.lay.n_blocks))
    xk_bits, xv_bits = bits16(li.xt_k), bits16(li.xt_v)
    for lo, hi in (calls or [(0, n_tok)]):
        B.twkv_compress(gc.h, layer, li.xt_k[lo:hi], li.xt_v[lo:hi], li.seq_ids[lo:hi], li.positions[lo:hi],
                        li.logits[lo:hi] if mode == B.TWKV_GATE_LOGITS else None, levels[lo:hi], mode)
        assert img.append(layer, xk_bits[lo:hi], xv_bits[lo:hi], seq_np[lo:hi], pos_np[lo:hi], ranks_np[lo:hi])
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    got_levels = levels.cpu().numpy().view(np.uint16).astype(np.int64)
    np.testing.assert_array_equal(got_levels, ranks_np)                      # per-token levels bit-exact
    if check_image:
        compare_cache_with_image(gc, img)
    st = B.twkv_cache_stats(gc.h, layer)
    assert st.tokens == n_tok and st.bytes_stored == img.stored_bytes(layer)
    assert st.bytes_algorithmic == int(2 * ranks_np.sum())
    assert abs(st.retain_rate_k - oracle.retain_rate(ranks_np[:, 0], li.d_kv)) < 1e-12
    assert abs(st.retain_rate_v - oracle.retain_rate(ranks_np[:, 1], li.d_kv)) < 1e-12
    # decode
    seqs = list(range(n_seq)) if decode_seqs is None else decode_seqs
    sid = torch.tensor(seqs, dtype=torch.int32, device="cuda")
    q = li.q[torch.as_tensor(seqs, device="cuda")].contiguous()
    out = torch.full((len(seqs), li.n_q_heads, 128), float("nan"), dtype=out_dtype, device="cuda")
    B.twkv_decode_attn(gc.h, layer, q, sid, out, num_splits)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    li_q = li.q
    li.q = q
    want = oracle_decode(li, ranks_np, seqs)
    li.q = li_q
    got = out.float().cpu().numpy()
    errs = attn_errors(got, want)
    gc.close()
    return errs, got, want


def test_config1_tiny_forced(B):
    # 1 sequence, 8 query heads = 8 KV heads, 1024 tokens, ranks uniform over {1024, 512, 256, 128}
    li = to_cuda(workloads.config(1))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), _, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_config1_fp16_output(B):
    li = to_cuda(workloads.config(1))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), _, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, out_dtype=torch.float16, check_image=False)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_any_rank_ragged_multi_call_gqa4(B):
    # 3 sequences of 301 tokens interleaved by the call pattern, every rank 1..1024, r_K != r_V,
    # compress in uneven calls including single-token appends; tiles end ragged (301 = 2 * 128 + 45)
    li = workloads.build_layer(11, n_seq=3, ctx=301, n_q_heads=32, mode="forced", rank_recipe="any", outlier="pct:1")
    g = torch.Generator().manual_seed(5)
    perm = torch.randperm(li.xt_k.shape[0], generator=g)                    # interleave the sequences
    for name in ["xt_k", "xt_v", "seq_ids", "positions", "ranks"]:
        setattr(li, name, getattr(li, name)[perm].contiguous())
    li = to_cuda(li)
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    n = ranks.shape[0]
    calls = [(0, 1), (1, 2), (2, 130), (130, 131), (131, 700), (700, n)]
    (max_abs, rel_l2), _, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, calls=calls, max_tokens_per_seq=400)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_logits_mode_levels_bit_exact_config2_shape(B):
    # config-2-shaped (GQA 4, gate-assigned ranks around 256), 2 sequences x 640 tokens
    li = workloads.config(2, ctx=640, n_seq=2)
    ranks, n_replaced = settle_logits(li.logits, 0.1, GATE_MARGIN_LOGITS)
    assert n_replaced < 0.05 * ranks.size
    li = to_cuda(li)
    (max_abs, rel_l2), _, _ = run_case(B, li, ranks.astype(np.int64), mode=B.TWKV_GATE_LOGITS)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    assert 150 < ranks.mean() < 400


def test_bf16_gqa8_long_recipe(B):
    # config-4-shaped: bf16, 64 query heads, sink + recent tokens at full rank, the rest 128 / 256
    li = to_cuda(workloads.config(4, ctx=1500))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    for splits in (0, 1, 3):
        (max_abs, rel_l2), _, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, num_splits=splits, check_image=splits == 0)
        assert max_abs < MAX_ABS and rel_l2 < REL_L2, (splits, max_abs, rel_l2)


def test_config3_shape_shuffled_positions_and_append(B):
    # skewed level mix, shuffled positions, 4 sequences x 200 tokens, then 5 decode-append steps
    li = workloads.config(3, ctx=205, n_seq=4)
    # reorder tokens so that the last 5 tokens of every sequence come last, one per sequence per step
    ctx, S = 205, 4
    idx = torch.arange(S * ctx).reshape(S, ctx)
    order = torch.cat([idx[:, :200].reshape(-1), idx[:, 200:].T.reshape(-1)])
    for name in ["xt_k", "xt_v", "seq_ids", "positions", "ranks"]:
        setattr(li, name, getattr(li, name)[order].contiguous())
    li = to_cuda(li)
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    calls = [(0, 800)] + [(800 + 4 * i, 804 + 4 * i) for i in range(5)]
    (max_abs, rel_l2), _, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, calls=calls)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_large_batch_of_short_sequences(B):
    # 37 sequences x 150 tokens: the merge kernel then takes two query slots per CTA (they share the reads of U_V^-1),
    # with a last group of one; the V pass runs with few splits per sequence
    li = to_cuda(workloads.config(3, ctx=150, n_seq=37))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), got, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED)
    assert np.all(np.isfinite(got))
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_long_context_full_size(B):
    # the long-context workload at its full size: one sequence of 131072 tokens, 64 query heads on 8 KV heads, bf16,
    # heavy-tailed outlier channels, full rank at the sink and the recent window and low rank between
    li = to_cuda(workloads.config(4))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), got, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED)
    assert np.all(np.isfinite(got))
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_high_batch_full_size_sampled(B):
    # the high-batch workload at its full size (64 sequences x 8192 tokens, shuffled positions, one compress call of
    # four pieces); the cache image is compared in full, the attention output on three sequences
    li = to_cuda(workloads.config(3))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), got, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, decode_seqs=[0, 41, 63])
    assert np.all(np.isfinite(got))
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_mixed_layer_workload_full_size_sampled(B):
    # one layer of the 32-layer decode workload at its full size (32 sequences x 16384 tokens, Dirichlet level mix);
    # levels and statistics on every token, the attention output on two sequences
    li = to_cuda(workloads.config(5))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), got, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, decode_seqs=[3, 30], check_image=False)
    assert np.all(np.isfinite(got))
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_tile_boundaries_and_single_token(B):
    for ctx in (1, 127, 128, 129):
        li = to_cuda(workloads.build_layer(20 + ctx, n_seq=2, ctx=ctx, n_q_heads=16, n_kv_heads=4, mode="forced",
                                           level_probs=(0.0, 0.0, 1.0, 0.0)))       # all tokens rank 256, one class
        li.ranks = li.ranks.clamp(max=li.d_kv)
        ranks = li.ranks.cpu().numpy().astype(np.int64)
        (max_abs, rel_l2), got, want = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED)
        assert max_abs < MAX_ABS and rel_l2 < REL_L2, (ctx, max_abs, rel_l2)


def test_rank_one_and_full_rank(B):
    li = to_cuda(workloads.build_layer(31, n_seq=1, ctx=200, n_q_heads=8, mode="forced"))
    ranks = np.ones((200, 2), dtype=np.int64)
    ranks[::3] = 1024
    ranks[1::7, 1] = 65
    (max_abs, rel_l2), _, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_one_split_over_more_tiles_than_the_v_pass_stages_at_once(B):
    # One sequence of 36 000 tokens (about 290 V tiles over four classes) decoded with a single split: the V pass stages
    # the tile descriptors of a split in shared memory 256 at a time, so this split crosses a refill; and with the
    # default split count (many short splits, some of them a single tile) the answer is the same within the bars.
    li = to_cuda(workloads.build_layer(47, n_seq=1, ctx=36000, n_q_heads=8, mode="forced", n_calib=2048))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    (max_abs, rel_l2), got1, want = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, num_splits=1, check_image=False)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    (max_abs, rel_l2), got0, _ = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, num_splits=0, check_image=False)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    assert np.abs(got1 - got0).max() < MAX_ABS


def test_subset_decode_empty_sequence_and_determinism(B):
    li = to_cuda(workloads.build_layer(41, n_seq=3, ctx=150, n_q_heads=32, mode="forced"))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    keep = (li.seq_ids != 1).cpu().numpy()                                   # sequence 1 stays empty
    sel = torch.from_numpy(np.nonzero(keep)[0]).cuda()
    for name in ["xt_k", "xt_v", "seq_ids", "positions"]:
        setattr(li, name, getattr(li, name)[sel].contiguous())
    ranks = ranks[keep]
    (e1, got1, _) = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, decode_seqs=[2, 0], max_tokens_per_seq=150)
    (e2, got2, _) = run_case(B, li, ranks, mode=B.TWKV_GATE_FORCED, decode_seqs=[2, 0], max_tokens_per_seq=150)
    assert e1[0] < MAX_ABS and e1[1] < REL_L2
    np.testing.assert_array_equal(got1, got2)                                # same inputs, same output bits
    # an empty sequence yields zeros
    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32,
                  max_seqs=3, max_tokens_per_seq=150, payload_bytes=1 << 20)
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k, li.Uinv_v)
    out = torch.full((1, 32, 128), 7.0, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q[:1].contiguous(), torch.tensor([1], dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    assert torch.count_nonzero(out).item() == 0
    gc.close()


def test_errors_leave_cache_unchanged(B):
    li = to_cuda(workloads.build_layer(51, n_seq=2, ctx=300, n_q_heads=32, mode="forced"))
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    n = ranks.shape[0]
    # pool with room for the tables but only 8 blocks of payload
    cfg = B.make_config(n_layers=1, n_q_heads=32, n_kv_heads=8, max_seqs=2, max_tokens_per_seq=300)
    tiny = B.twkv_cache_required_bytes(cfg, 0) - (1 * 2 * 2 * 136) * 16384 + 8 * 16384   # drop the slack blocks
    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32,
                  max_seqs=2, max_tokens_per_seq=300, payload_bytes=0, pool_bytes=tiny)
    assert int(gc.lay.n_blocks) == 8
    lv = levels_tensor(ranks)
    B.twkv_compress(gc.h, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, lv, B.TWKV_GATE_FORCED)
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_CAPACITY
    t = gc.tables()
    assert t["status"][1] == 0 and t["n_tiles"].sum() == 0 and t["fill"].sum() == 0
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK                          # sticky status was cleared by the read
    gc.close()
    # invalid rank, sequence id, position; too many tokens for one sequence; duplicate decode ids
    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32,
                  max_seqs=2, max_tokens_per_seq=299, payload_bytes=64 << 20)
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k, li.Uinv_v)
    B.twkv_compress(gc.h, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, lv, B.TWKV_GATE_FORCED)
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_CAPACITY              # 300 tokens > 299 per sequence
    for what in ("rank0", "rank_big", "seq", "pos"):
        bad_lv, bad_seq, bad_pos = lv.clone(), li.seq_ids.clone(), li.positions.clone()
        if what == "rank0": bad_lv[5, 1] = 0
        if what == "rank_big": bad_lv[5, 0] = 1025
        if what == "seq": bad_seq[7] = 2
        if what == "pos": bad_pos[9] = -1
        B.twkv_compress(gc.h, 0, li.xt_k[:100], li.xt_v[:100], bad_seq[:100], bad_pos[:100], None, bad_lv[:100], B.TWKV_GATE_FORCED)
        assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_INVALID_ARG, what
        assert gc.tables()["fill"].sum() == 0
    out = torch.zeros(2, 32, 128, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q, torch.tensor([1, 1], dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_INVALID_ARG
    # host-side argument errors
    with pytest.raises(B.TwkvError):
        B.twkv_compress(gc.h, 3, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, lv, B.TWKV_GATE_FORCED)
    with pytest.raises(B.TwkvError):
        B.twkv_compress(gc.h, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, lv, B.TWKV_GATE_LOGITS)
    with pytest.raises(B.TwkvError):
        B.twkv_decode_attn(gc.h, 0, li.q, torch.tensor([0, 1], dtype=torch.int32, device="cuda"), out, num_splits=100000)
    gc.close()


def test_two_layers_share_one_pool(B):
    li0 = to_cuda(workloads.build_layer(61, n_seq=2, ctx=140, n_q_heads=32, mode="forced"))
    li1 = to_cuda(workloads.build_layer(62, n_seq=2, ctx=140, n_q_heads=32, mode="forced", rank_recipe="any"))
    r0, r1 = li0.ranks.cpu().numpy().astype(np.int64), li1.ranks.cpu().numpy().astype(np.int64)
    payload = int((-(-r0 // 64) * 128).sum() + (-(-r1 // 64) * 128).sum())
    gc = GpuCache(B, n_layers=2, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32,
                  max_seqs=2, max_tokens_per_seq=140, payload_bytes=payload)
    img = CacheImage(2, 1024, 2, 140, int(gc.lay.n_blocks))
    for l, (li, r) in enumerate(((li0, r0), (li1, r1))):
        B.twkv_cache_set_layer_params(gc.h, l, li.Uinv_k, li.Uinv_v)
    # interleave the layers' compress calls
    for lo, hi in ((0, 100), (100, 280)):
        for l, (li, r) in enumerate(((li0, r0), (li1, r1))):
            B.twkv_compress(gc.h, l, li.xt_k[lo:hi], li.xt_v[lo:hi], li.seq_ids[lo:hi], li.positions[lo:hi], None,
                            levels_tensor(r[lo:hi]), B.TWKV_GATE_FORCED)
            assert img.append(l, bits16(li.xt_k[lo:hi]), bits16(li.xt_v[lo:hi]), li.seq_ids[lo:hi].cpu().numpy(),
                              li.positions[lo:hi].cpu().numpy(), r[lo:hi])
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    compare_cache_with_image(gc, img)
    sid = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    for l, (li, r) in enumerate(((li0, r0), (li1, r1))):
        out = torch.empty(2, 32, 128, device="cuda")
        B.twkv_decode_attn(gc.h, l, li.q, sid, out)
        max_abs, rel_l2 = attn_errors(out.cpu().numpy(), oracle_decode(li, r, [0, 1]))
        assert max_abs < MAX_ABS and rel_l2 < REL_L2, (l, max_abs, rel_l2)
    st = B.twkv_cache_stats(gc.h, -1)
    assert st.tokens == 560 and st.blocks_used == img.next_block
    # reset forgets everything
    B.twkv_cache_reset(gc.h)
    assert gc.tables()["fill"].sum() == 0 and B.twkv_cache_stats(gc.h, -1).tokens == 0
    gc.close()


def _compute_mode_case(B, *, n_kv_heads, n_q_heads, dtype, ctx, n_seq, seed, li=None, gate_seed=None, calls=None,
                       max_loose=0.05):
    """COMPUTE-mode compress + decode against the oracle.  The library forms z = x~ W + b itself (calls of 1024 tokens or
    more: the fused tcgen05 gate; smaller calls: the warp-MMA GEMM + the rank kernel).  Every token is checked
    (check_gate_levels): bit-exact rank wherever the oracle's decision has a relative margin of GATE_MARGIN_COMPUTE,
    otherwise a rank inside the interval the margin allows.  The cache image and the attention output are then
    compared with the oracle run on the validated ranks."""
    from tests.helpers import GATE_MARGIN_COMPUTE, check_gate_levels
    dn = "f16" if dtype == torch.float16 else "bf16"
    if li is None:
        li = workloads.build_layer(seed, n_seq=n_seq, ctx=ctx, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, dtype=dtype,
                                   outlier="pct:1", mode="forced")
    d = li.d_kv
    Wk, Wv, bk, bv = workloads.gate_params(seed + 1 if gate_seed is None else gate_seed, d, dtype, n_bumps=min(64, d // 4),
                                           first_dim=min(64, d // 4))
    zk = oracle.gate_logits(oracle.widen16(bits16(li.xt_k), dn), oracle.widen16(bits16(Wk), dn), bk.double().numpy())
    zv = oracle.gate_logits(oracle.widen16(bits16(li.xt_v), dn), oracle.widen16(bits16(Wv), dn), bv.double().numpy())
    li = to_cuda(li)
    n = li.xt_k.shape[0]
    seq_np, pos_np = li.seq_ids.cpu().numpy(), li.positions.cpu().numpy()
    tmax = int(np.bincount(seq_np, minlength=n_seq).max())
    gc = GpuCache(B, n_layers=1, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, dtype=dtype, out_dtype=torch.float32,
                  max_seqs=n_seq, max_tokens_per_seq=tmax, payload_bytes=n * 4 * d)
    gate = [t.cuda().contiguous() for t in (Wk, Wv, bk, bv)]       # borrowed by the cache: keep them alive
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k, li.Uinv_v, *gate)
    levels = torch.zeros(n, 2, dtype=torch.int16, device="cuda")
    for lo, hi in (calls or [(0, n)]):
        B.twkv_compress(gc.h, 0, li.xt_k[lo:hi], li.xt_v[lo:hi], li.seq_ids[lo:hi], li.positions[lo:hi], None, levels[lo:hi],
                        B.TWKV_GATE_COMPUTE)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    ranks = levels.cpu().numpy().view(np.uint16).astype(np.int64)
    n_loose = check_gate_levels(ranks, zk, zv, 0.1, GATE_MARGIN_COMPUTE)
    assert n_loose <= max_loose * 2 * n + 2, (n_loose, n)
    img = CacheImage(1, d, n_seq, tmax, int(gc.lay.n_blocks))
    xk_bits, xv_bits = bits16(li.xt_k), bits16(li.xt_v)
    for lo, hi in (calls or [(0, n)]):
        assert img.append(0, xk_bits[lo:hi], xv_bits[lo:hi], seq_np[lo:hi], pos_np[lo:hi], ranks[lo:hi])
    compare_cache_with_image(gc, img)
    seqs = list(range(n_seq))
    out = torch.empty(n_seq, n_q_heads, 128, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q, torch.tensor(seqs, dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    errs = attn_errors(out.cpu().numpy(), oracle_decode(li, ranks, seqs))
    gc.close()
    return errs, ranks, n_loose


def test_compute_mode_gate_levels_bit_exact(B):
    # config-2-shaped states, 2 x 700 tokens in one call: the fused tcgen05 gate
    li = workloads.config(2, ctx=700, n_seq=2)
    (max_abs, rel_l2), ranks, n_loose = _compute_mode_case(B, n_kv_heads=8, n_q_heads=32, dtype=torch.float16, ctx=700, n_seq=2,
                                                           seed=0, li=li, gate_seed=7)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    assert len(np.unique(ranks)) > 20


@pytest.mark.parametrize("n_tok", [1, 64, 129, 1023])
@pytest.mark.parametrize("dtype,n_kv_heads,n_q_heads", [(torch.float16, 8, 32), (torch.bfloat16, 8, 64), (torch.float16, 3, 6)])
def test_compute_mode_small_calls(B, n_tok, dtype, n_kv_heads, n_q_heads):
    # calls of fewer than 1024 tokens (the decode-time append) take the warp-MMA logits GEMM and the warp-per-row rank
    # kernel instead of the fused gate: ranks, cache image and attention against the oracle, d_kv = 1024 and 384
    n_seq = 1 if n_tok < 4 else 2
    ctx = -(-n_tok // n_seq)
    li = workloads.build_layer(300 + n_tok, n_seq=n_seq, ctx=ctx, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, dtype=dtype,
                               outlier="pct:1", mode="forced", n_calib=2048)
    if n_seq * ctx > n_tok:                                              # odd token count: drop the last token
        for name in ["xt_k", "xt_v", "seq_ids", "positions"]:
            setattr(li, name, getattr(li, name)[:n_tok].contiguous())
    (max_abs, rel_l2), ranks, _ = _compute_mode_case(B, n_kv_heads=n_kv_heads, n_q_heads=n_q_heads, dtype=dtype, ctx=ctx,
                                                     n_seq=n_seq, seed=300 + n_tok, li=li)
    assert ranks.shape[0] == n_tok
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_compute_mode_prefill_then_appends(B):
    # one prefill call through the fused gate, then single-token-per-sequence appends through the small-call gate:
    # both paths fill one cache, every token's rank is checked against the oracle
    n_seq, ctx = 2, 640
    li = workloads.build_layer(333, n_seq=n_seq, ctx=ctx + 4, n_q_heads=32, dtype=torch.float16, outlier="pct:1", mode="forced")
    idx = torch.arange(n_seq * (ctx + 4)).reshape(n_seq, ctx + 4)
    order = torch.cat([idx[:, :ctx].reshape(-1), idx[:, ctx:].T.reshape(-1)])
    for name in ["xt_k", "xt_v", "seq_ids", "positions"]:
        setattr(li, name, getattr(li, name)[order].contiguous())
    calls = [(0, n_seq * ctx)] + [(n_seq * ctx + n_seq * i, n_seq * ctx + n_seq * (i + 1)) for i in range(4)]
    (max_abs, rel_l2), _, _ = _compute_mode_case(B, n_kv_heads=8, n_q_heads=32, dtype=torch.float16, ctx=ctx + 4, n_seq=n_seq,
                                                 seed=333, li=li, calls=calls)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_compute_mode_bf16_four_kv_heads(B):
    # d_kv = 512 (two 256-wide logit slabs), bf16, GQA 8, a ragged 1300-token call
    (max_abs, rel_l2), ranks, _ = _compute_mode_case(B, n_kv_heads=4, n_q_heads=32, dtype=torch.bfloat16, ctx=650, n_seq=2, seed=71)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    assert ranks.min() >= 1 and ranks.max() <= 512


def test_compute_mode_three_kv_heads(B):
    # d_kv = 384: 128-wide logit slabs in the gate, an odd number of KV-head slabs in the K-score kernel, GQA 2
    (max_abs, rel_l2), _, _ = _compute_mode_case(B, n_kv_heads=3, n_q_heads=6, dtype=torch.float16, ctx=600, n_seq=2, seed=73)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)


def test_compress_spanning_two_pieces(B):
    # one call of 131072 + 300 tokens is processed as two pieces; levels, tables and packed bytes must still match
    # the oracle's image (small ranks keep the case light), and decode must agree on one of the sequences
    n_seq, ctx = 4, 32843
    li = workloads.build_layer(81, n_seq=n_seq, ctx=ctx, n_q_heads=8, mode="forced", level_probs=(0.0, 0.0, 0.02, 0.98),
                               n_calib=2048)
    assert li.xt_k.shape[0] > B.PIECE_TOKENS
    li = to_cuda(li)
    ranks = li.ranks.cpu().numpy().astype(np.int64)
    gc = GpuCache(B, n_layers=1, n_q_heads=8, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32,
                  max_seqs=n_seq, max_tokens_per_seq=ctx, payload_bytes=int((-(-ranks // 64) * 128).sum()))
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k, li.Uinv_v)
    B.twkv_compress(gc.h, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, levels_tensor(ranks), B.TWKV_GATE_FORCED)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    img = CacheImage(1, li.d_kv, n_seq, ctx, int(gc.lay.n_blocks))
    assert img.append(0, bits16(li.xt_k), bits16(li.xt_v), li.seq_ids.cpu().numpy(), li.positions.cpu().numpy(), ranks)
    compare_cache_with_image(gc, img)
    out = torch.empty(1, 8, 128, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q[3:4].contiguous(), torch.tensor([3], dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    li_q = li.q
    li.q = li.q[3:4]
    want = oracle_decode(li, ranks, [3])
    li.q = li_q
    max_abs, rel_l2 = attn_errors(out.cpu().numpy(), want)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    gc.close()


def test_three_pieces_middle_one_refused(B):
    # One call of three pieces whose bookkeeping is launched together.  The middle piece would push sequence 0 past
    # max_tokens_per_seq: it is skipped whole (sticky TWKV_ERR_CAPACITY), the pieces before and after it are stored, and
    # the third one continues the tiles of nothing the refused piece touched.
    P = B.PIECE_TOKENS
    half, tmax, d = P // 2, 70000, 1024
    seq = torch.cat([torch.full((half,), 0), torch.full((half,), 1), torch.full((half,), 0), torch.full((half,), 2),
                     torch.full((500,), 2)]).to(torch.int32)
    n = seq.numel()
    pos = torch.zeros(n, dtype=torch.int32)
    for s_ in range(3):
        m = seq == s_
        pos[m] = torch.arange(int(m.sum()), dtype=torch.int32)
    g = torch.Generator().manual_seed(91)
    xk = (torch.randn(n, d, generator=g) * 0.5).to(torch.float16)
    xv = (torch.randn(n, d, generator=g) * 0.5).to(torch.float16)
    ranks = torch.randint(1, 129, (n, 2), generator=g).numpy().astype(np.int64)        # classes 1 and 2 keep the case light
    gc = GpuCache(B, n_layers=1, n_q_heads=8, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32,
                  max_seqs=3, max_tokens_per_seq=tmax, payload_bytes=int((-(-ranks // 64) * 128).sum()))
    U = torch.eye(d, dtype=torch.float16).cuda()
    B.twkv_cache_set_layer_params(gc.h, 0, U, U)
    B.twkv_compress(gc.h, 0, xk.cuda(), xv.cuda(), seq.cuda(), pos.cuda(), None, levels_tensor(ranks), B.TWKV_GATE_FORCED)
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_CAPACITY                            # read once: cleared
    img = CacheImage(1, d, 3, tmax, int(gc.lay.n_blocks))
    got = []
    for lo in range(0, n, P):                                                           # the image takes the pieces one by one
        hi = min(n, lo + P)
        got.append(img.append(0, bits16(xk[lo:hi]), bits16(xv[lo:hi]), seq[lo:hi].numpy(), pos[lo:hi].numpy(), ranks[lo:hi]))
    assert got == [True, False, True]
    compare_cache_with_image(gc, img)
    st = B.twkv_cache_stats(gc.h, 0)
    assert st.tokens == P + 500
    gc.close()


def test_benchmark_workload_full_size_sampled(B):
    # the workload and launch configuration bench.py times (B = 16, T = 32768, GQA 4, fp16, COMPUTE gate), checked
    # on what the oracle can afford: the ranks of every token of one sequence, and that sequence's attention output
    import bench
    dev = torch.device("cuda", 0)
    li, gate = bench.build_workload(dev)
    Wk, Wv, bk, bv = gate
    n_seq, ctx, Hq = bench.B_SEQ, bench.CTX, bench.HQ
    n_tok = n_seq * ctx
    cfg = B.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=bench.HKV, dtype=torch.float16, out_dtype=torch.float32,
                        max_seqs=n_seq, max_tokens_per_seq=ctx)
    pool = torch.empty(B.twkv_cache_required_bytes(cfg, int(n_tok * 2 * 2 * 420)), dtype=torch.uint8, device=dev)
    cache = B.twkv_cache_create(cfg, pool)
    B.twkv_cache_set_layer_params(cache, 0, li.Uinv_k, li.Uinv_v, Wk, Wv, bk, bv)
    levels = torch.zeros(n_tok, 2, dtype=torch.int16, device=dev)
    B.twkv_compress(cache, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, levels, B.TWKV_GATE_COMPUTE)
    out = torch.empty(n_seq, Hq, 128, dtype=torch.float32, device=dev)
    B.twkv_decode_attn(cache, 0, li.q, torch.arange(n_seq, dtype=torch.int32, device=dev), out)
    assert B.twkv_cache_status(cache) == B.TWKV_OK
    st = B.twkv_cache_stats(cache, 0)
    got = levels.cpu().numpy().view(np.uint16).astype(np.int64)
    assert st.tokens == n_tok and st.bytes_algorithmic == int(2 * got.sum())
    s = 5                                                                 # the sampled sequence
    lo, hi = s * ctx, (s + 1) * ctx
    xk = oracle.widen16(bits16(li.xt_k[lo:hi]), "f16")
    xv = oracle.widen16(bits16(li.xt_v[lo:hi]), "f16")
    from tests.helpers import GATE_MARGIN_COMPUTE, check_gate_levels
    zk = oracle.gate_logits(xk, oracle.widen16(bits16(Wk), "f16"), bk.double().cpu().numpy())
    zv = oracle.gate_logits(xv, oracle.widen16(bits16(Wv), "f16"), bv.double().cpu().numpy())
    n_loose = check_gate_levels(got[lo:hi], zk, zv, 0.1, GATE_MARGIN_COMPUTE)
    assert n_loose < 0.02 * 2 * ctx, n_loose
    # attention of the sampled sequence, with the ranks the library assigned (they equal the oracle's wherever the
    # oracle's decision does not hinge on rounding)
    want = oracle.decode_attn(xk, xv, got[lo:hi, 0], got[lo:hi, 1], li.positions[lo:hi].cpu().numpy(),
                              oracle.widen16(bits16(li.Uinv_k), "f16"), oracle.widen16(bits16(li.Uinv_v), "f16"),
                              oracle.widen16(bits16(li.q[s]), "f16"), bench.HKV, 500000.0, 128 ** -0.5)
    max_abs, rel_l2 = attn_errors(out[s].cpu().numpy(), want)
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    B.twkv_cache_destroy(cache)
