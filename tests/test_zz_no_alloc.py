"""twkv_gate_ranks_static: the allocation-free gate entry point.

Some callers need a token's ranks at a moment when they cannot obtain device memory (no cache
pool yet, or a framework that owns the whole device and forbids allocations).  This entry point
stages its logits in a fixed array inside the library instead.  The test calls it through the C
ABI twice in a row, on different tokens, and checks every rank against the CPU oracle's gate
(Eq. 5, 6, 8) under the rule all COMPUTE-mode tests use: bit-exact where the oracle's decision has
a relative margin of 1e-3, inside the interval that margin allows otherwise.  It also compares it
with the pool-backed path (twkv_compress in TWKV_GATE_COMPUTE mode, here the fused tensor-core
gate): the two evaluate the same formulas in fp32 in different orders, so they must agree bit for
bit wherever the decision is not within rounding of tau.  It lives in the last-collected file so
that a run stopping at the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_04411_b200 import workloads

pytestmark = pytest.mark.gpu


def test_static_gate_matches_pool_backed_gate_twice():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    from tests.helpers import GATE_MARGIN_COMPUTE, GpuCache, bits16, check_gate_levels

    li = workloads.config(2, ctx=512, n_seq=2)
    gate_cpu = workloads.gate_params(3, li.d_kv, torch.float16)
    w = lambda t: oracle.widen16(bits16(t), "f16")
    zk = oracle.gate_logits(w(li.xt_k), w(gate_cpu[0]), gate_cpu[2].double().numpy())
    zv = oracle.gate_logits(w(li.xt_v), w(gate_cpu[1]), gate_cpu[3].double().numpy())
    safe = np.stack([oracle.gate_rank(zk, 0.1)[1], oracle.gate_rank(zv, 0.1)[1]], axis=1) >= GATE_MARGIN_COMPUTE
    Wk, Wv, bk, bv = [t.cuda().contiguous() for t in gate_cpu]
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
    check_gate_levels(want, zk, zv, 0.1, GATE_MARGIN_COMPUTE)

    # two calls in a row on different token ranges: the second must not see the first one's logits
    for lo, hi in ((0, 512), (512, 1024)):
        got = torch.full((hi - lo, 2), -1, dtype=torch.int16, device="cuda")
        B.twkv_gate_ranks_static(xk[lo:hi], xv[lo:hi], Wk, Wv, bk, bv, got)
        torch.cuda.synchronize()
        got = got.cpu().numpy().view(np.uint16)
        check_gate_levels(got, zk[lo:hi], zv[lo:hi], 0.1, GATE_MARGIN_COMPUTE)
        np.testing.assert_array_equal(got[safe[lo:hi]], want[lo:hi][safe[lo:hi]])
    # a short call after a long one, and the size limit
    got = torch.zeros(7, 2, dtype=torch.int16, device="cuda")
    B.twkv_gate_ranks_static(xk[100:107], xv[100:107], Wk, Wv, bk, bv, got)
    check_gate_levels(got.cpu().numpy().view(np.uint16), zk[100:107], zv[100:107], 0.1, GATE_MARGIN_COMPUTE)
    too_many = torch.zeros(513, 2, dtype=torch.int16, device="cuda")
    with pytest.raises(B.TwkvError) as err:
        B.twkv_gate_ranks_static(xk[:513], xv[:513], Wk, Wv, bk, bv, too_many)
    assert err.value.code == B.TWKV_ERR_CAPACITY
    gc.close()
