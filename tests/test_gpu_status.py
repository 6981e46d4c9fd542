"""Status codes that only the device can raise, provoked from the host (nothing here faults, traps or hangs a GPU).

* TWKV_ERR_TIMEOUT: the bounded wait of the tensor-core kernels, run on a barrier nobody completes with a small
  attempt limit, gives up, raises its flag and reports the code; the cache keeps working afterwards.
* TWKV_ERR_DEVICE_CHECK: twkv_cache_check finds a guard word or a table entry that the host has overwritten.
"""
import numpy as np
import pytest
import torch

from paper_2603_04411_b200 import workloads
from tests.helpers import GpuCache

pytestmark = pytest.mark.gpu


def _filled_cache(B):
    li = workloads.build_layer(950, n_seq=2, ctx=300, n_q_heads=32, mode="forced", rank_recipe="any")
    ranks = li.ranks.numpy().astype(np.int64)
    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32, max_seqs=2,
                  max_tokens_per_seq=300, payload_bytes=int((-(-ranks // 64) * 128).sum()))
    gc.layer_params = (li.Uinv_k.cuda(), li.Uinv_v.cuda())              # borrowed by the cache: they must outlive it
    B.twkv_cache_set_layer_params(gc.h, 0, *gc.layer_params)
    B.twkv_compress(gc.h, 0, li.xt_k.cuda(), li.xt_v.cuda(), li.seq_ids.cuda(), li.positions.cuda(), None,
                    torch.from_numpy(ranks.astype(np.int16)).cuda(), B.TWKV_GATE_FORCED)
    return gc, li


def _decode(B, gc, li):
    out = torch.empty(2, 32, 128, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q.cuda(), torch.tensor([0, 1], dtype=torch.int32, device="cuda"), out)
    return out


def test_bounded_wait_gives_up_and_the_cache_keeps_working():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    gc, li = _filled_cache(B)
    before = _decode(B, gc, li)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    times = []
    for attempts in (64, 1024, 16384):
        code, ns = B.twkv_selftest_wait_timeout(gc.h, attempts)
        assert code == B.TWKV_OK, "the wait did not give up"
        assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_TIMEOUT            # reported once, like a production timeout
        assert B.twkv_cache_status(gc.h) == B.TWKV_OK
        times.append(ns)
    print("bounded wait, nanoseconds for 64 / 1024 / 16384 attempts:", times)
    assert times[2] > times[0]
    after = _decode(B, gc, li)                                              # the next production call is unaffected
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    torch.testing.assert_close(after, before, rtol=0, atol=0)
    gc.close()


def test_cache_check_finds_overwritten_guards_and_tables():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    gc, li = _filled_cache(B)
    _decode(B, gc, li)
    assert B.twkv_cache_check(gc.h, -1) == (B.TWKV_OK, 0)
    lay = gc.lay
    NT = int(lay.max_tiles)
    # a stored rank outside its tile's class
    off = int(lay.tile_rank_off)
    saved = gc.pool[off:off + 2].clone()
    gc.pool[off:off + 2] = torch.tensor([0xFF, 0x7F], dtype=torch.uint8, device="cuda")
    code, bad = B.twkv_cache_check(gc.h, 0)
    assert code == B.TWKV_ERR_DEVICE_CHECK and bad >= 1
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_DEVICE_CHECK
    gc.pool[off:off + 2] = saved
    assert B.twkv_cache_check(gc.h, 0) == (B.TWKV_OK, 0)
    # a V slot linked past the K tiles
    off = int(lay.tile_aux_off) + NT * 128 * 4
    saved = gc.pool[off:off + 4].clone()
    gc.pool[off:off + 4] = torch.tensor([0xFF, 0xFF, 0xFF, 0x3F], dtype=torch.uint8, device="cuda")
    assert B.twkv_cache_check(gc.h, 0)[0] == B.TWKV_ERR_DEVICE_CHECK
    gc.pool[off:off + 4] = saved
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_DEVICE_CHECK
    # the guard word behind the status block (a write that ran over the end of a region)
    saved = gc.pool[32:40].clone()
    gc.pool[32:40] = 0
    code, bad = B.twkv_cache_check(gc.h, 0)
    assert code == B.TWKV_ERR_DEVICE_CHECK and bad == 1
    gc.pool[32:40] = saved
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_DEVICE_CHECK
    assert B.twkv_cache_check(gc.h, -1) == (B.TWKV_OK, 0)
    # a reset keeps the guards
    B.twkv_cache_reset(gc.h)
    assert B.twkv_cache_check(gc.h, -1) == (B.TWKV_OK, 0)
    gc.close()


def test_non_finite_logits_and_out_of_range_values_are_reported():
    import os
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    # (1) LOGITS mode with a NaN and an infinite logit: the call reports TWKV_ERR_DEVICE_CHECK (ranks are placeholders)
    li = workloads.config(2, ctx=64, n_seq=1)
    logits = li.logits.clone()
    logits[5, 0, 17] = float("nan")
    logits[9, 1, 3] = float("inf")
    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float32, max_seqs=1,
                  max_tokens_per_seq=64, payload_bytes=64 * 4096)
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k.cuda(), li.Uinv_v.cuda())
    lv = torch.zeros(64, 2, dtype=torch.int16, device="cuda")
    B.twkv_compress(gc.h, 0, li.xt_k.cuda(), li.xt_v.cuda(), li.seq_ids.cuda(), li.positions.cuda(), logits.cuda(), lv, B.TWKV_GATE_LOGITS)
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_DEVICE_CHECK
    got = lv.cpu().numpy().view(np.uint16)
    assert got.min() >= 1 and got.max() <= 1024                            # still inside the valid range
    gc.close()
    # (2) a bf16 query beyond the f16 range
    li = workloads.build_layer(960, n_seq=1, ctx=100, n_q_heads=64, dtype=torch.bfloat16, mode="forced")
    ranks = li.ranks.numpy().astype(np.int64)

    def run(q, xk_scale=1.0):
        gc = GpuCache(B, n_layers=1, n_q_heads=64, n_kv_heads=8, dtype=torch.bfloat16, out_dtype=torch.float32, max_seqs=1,
                      max_tokens_per_seq=100, payload_bytes=int((-(-ranks // 64) * 128).sum()))
        B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k.cuda(), li.Uinv_v.cuda())
        B.twkv_compress(gc.h, 0, (li.xt_k.float() * xk_scale).to(torch.bfloat16).cuda(), li.xt_v.cuda(), li.seq_ids.cuda(),
                        li.positions.cuda(), None, torch.from_numpy(ranks.astype(np.int16)).cuda(), B.TWKV_GATE_FORCED)
        out = torch.empty(1, 64, 128, device="cuda")
        B.twkv_decode_attn(gc.h, 0, q.cuda().contiguous(), torch.tensor([0], dtype=torch.int32, device="cuda"), out)
        code = B.twkv_cache_status(gc.h)
        gc.close()
        return code
    assert run(li.q) == B.TWKV_OK
    big = li.q.clone(); big[0, 7, 100] = 1.0e6
    assert run(big) == B.TWKV_ERR_DEVICE_CHECK
    # (3) rotated keys beyond the f16 range: clamped silently by default, reported with TWKV_DEBUG=1
    assert run(li.q, xk_scale=3.0e4) == B.TWKV_OK
    os.environ["TWKV_DEBUG"] = "1"
    try:
        assert run(li.q, xk_scale=3.0e4) == B.TWKV_ERR_DEVICE_CHECK
        assert run(li.q) == B.TWKV_OK
    finally:
        del os.environ["TWKV_DEBUG"]


def test_decode_query_with_a_sequence_id_outside_the_cache_gets_zeros():
    """The header's promise for an id the host cannot check against anything (ids live in device memory): the code
    is reported, that query's output is defined (zeros), the other query's output is what it is without the bad one."""
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    gc, li = _filled_cache(B)
    good = _decode(B, gc, li)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    out = torch.full((2, 32, 128), 7.0, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q.cuda(), torch.tensor([0, 99], dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_ERR_INVALID_ARG
    assert torch.count_nonzero(out[1]).item() == 0
    torch.testing.assert_close(out[0], good[0], rtol=0, atol=0)
    again = _decode(B, gc, li)                                              # and the cache is as it was
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    torch.testing.assert_close(again, good, rtol=0, atol=0)
    gc.close()


def test_decode_call_replays_from_a_cuda_graph():
    """A decode call enqueues kernels only (no allocation, no synchronisation, no host-side reads of device state), so a
    captured call can be replayed: the replay's output equals the eager call's bit for bit."""
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    gc, li = _filled_cache(B)
    eager = _decode(B, gc, li)                                              # also the first call's one-time set-up
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    q = li.q.cuda()
    sid = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    out = torch.zeros(2, 32, 128, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.twkv_decode_attn(gc.h, 0, q, sid, out)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        torch.testing.assert_close(out, eager, rtol=0, atol=0)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    gc.close()
