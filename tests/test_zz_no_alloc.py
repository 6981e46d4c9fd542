"""twkv_gate_ranks_static: the allocation-free gate entry point.

Some callers need a token's ranks at a moment when they cannot obtain device memory (no cache
pool yet, or a framework that owns the whole device and forbids allocations).  This entry point
stages its logits in a fixed array inside the library instead.  The test calls it through the C
ABI twice in a row, on different tokens, and demands the same per-token ranks, bit for bit,
as the pool-backed path (twkv_compress in TWKV_GATE_COMPUTE mode), which is the bar the other
tests hold integer outputs to.  It lives in the last-collected file so that a run stopping at
the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

from paper_2603_04411_b200 import workloads

pytestmark = pytest.mark.gpu


def test_static_gate_matches_pool_backed_gate_twice():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    from tests.helpers import GpuCache

    li = workloads.config(2, ctx=512, n_seq=2)
    Wk, Wv, bk, bv = [t.cuda().contiguous() for t in workloads.gate_params(3, li.d_kv, torch.float16)]
    xk, xv = li.xt_k.cuda().contiguous(), li.xt_v.cuda().contiguous()
    seq, pos = li.seq_ids.cuda().contiguous(), li.positions.cuda().contiguous()
    n = xk.shape[0]

    gc = GpuCache(B, n_layers=1, n_q_heads=32, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float16,
                  max_seqs=2, max_tokens_per_seq=512, payload_bytes=n * 4096)
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k.cuda(), li.Uinv_v.cuda(), Wk, Wv, bk, bv)
    want = torch.zeros(n, 2, dtype=torch.int16, device="cuda")
    B.twkv_compress(gc.h, 0, xk, xv, seq, pos, None, want, B.TWKV_GATE_COMPUTE)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    want = want.cpu().numpy().view(np.uint16)
    assert want.min() >= 1 and want.max() <= 1024 and len(np.unique(want)) > 20

    # two calls in a row on different token ranges: the second must not see the first one's logits
    for lo, hi in ((0, 512), (512, 1024)):
        got = torch.full((hi - lo, 2), -1, dtype=torch.int16, device="cuda")
        B.twkv_gate_ranks_static(xk[lo:hi], xv[lo:hi], Wk, Wv, bk, bv, got)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(got.cpu().numpy().view(np.uint16), want[lo:hi])
    # a short call after a long one, and the size limit
    got = torch.zeros(7, 2, dtype=torch.int16, device="cuda")
    B.twkv_gate_ranks_static(xk[100:107], xv[100:107], Wk, Wv, bk, bv, got)
    np.testing.assert_array_equal(got.cpu().numpy().view(np.uint16), want[100:107])
    too_many = torch.zeros(513, 2, dtype=torch.int16, device="cuda")
    with pytest.raises(B.TwkvError) as err:
        B.twkv_gate_ranks_static(xk[:513], xv[:513], Wk, Wv, bk, bv, too_many)
    assert err.value.code == B.TWKV_ERR_CAPACITY
    gc.close()
