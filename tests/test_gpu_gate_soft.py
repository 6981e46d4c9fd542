"""GPU parity of the soft gate (twkv_gate_soft: Eq. 6, Eq. 7, soft Retain Rate) against the CPU oracle.

Tolerance: the library forms the logits in fp32 from exact 16-bit products (error below 1e-4 absolute for |z| of a few
tens) and evaluates softmax and cumulative sums in fp32, so every cumulative sum m_i in [0, 1] is within 2e-4 of the
fp64 value; x~ (.) m inherits that times |x~|.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_04411_b200 import workloads
from tests.helpers import GpuCache, bits16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,n_kv_heads,n_tok", [(torch.float16, 8, 700), (torch.bfloat16, 3, 129), (torch.float16, 8, 9000)])
def test_soft_gate_matches_oracle(dtype, n_kv_heads, n_tok):
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    dn = "f16" if dtype == torch.float16 else "bf16"
    li = workloads.build_layer(900 + n_tok, n_seq=1, ctx=n_tok, n_q_heads=n_kv_heads, n_kv_heads=n_kv_heads, dtype=dtype,
                               outlier="pct:1", mode="forced", n_calib=2048)
    d = li.d_kv
    Wk, Wv, bk, bv = workloads.gate_params(901, d, dtype, n_bumps=min(64, d // 4), first_dim=min(64, d // 4))
    w = lambda t: oracle.widen16(bits16(t), dn)
    want = {}
    for side, x, W, b in (("k", li.xt_k, Wk, bk), ("v", li.xt_v, Wv, bv)):
        z = oracle.gate_logits(w(x), w(W), b.double().numpy())
        want[side] = oracle.soft_gate(w(x), z)
    gc = GpuCache(B, n_layers=1, n_q_heads=n_kv_heads, n_kv_heads=n_kv_heads, dtype=dtype, out_dtype=torch.float32, max_seqs=1,
                  max_tokens_per_seq=n_tok, payload_bytes=1 << 20)
    params = [t.cuda().contiguous() for t in (li.Uinv_k, li.Uinv_v, Wk, Wv, bk, bv)]
    B.twkv_cache_set_layer_params(gc.h, 0, *params)
    xk, xv = li.xt_k.cuda().contiguous(), li.xt_v.cuda().contiguous()
    m_k, m_v, xh_k, xh_v = (torch.full((n_tok, d), float("nan"), device="cuda") for _ in range(4))
    ret = torch.full((n_tok, 2), float("nan"), device="cuda")
    B.twkv_gate_soft(gc.h, 0, xk, xv, m_k, m_v, xh_k, xh_v, ret)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    for side, m, xh, col in (("k", m_k, xh_k, 0), ("v", m_v, xh_v, 1)):
        om, oxh, oR = want[side]
        gm = m.cpu().numpy().astype(np.float64)
        assert np.abs(gm - om).max() < 2e-4
        assert np.all(np.diff(gm, axis=1) <= 1e-6) and np.abs(gm[:, 0] - 1).max() < 1e-5      # non-increasing, m_1 = 1
        scale = np.abs(w(li.xt_k if side == "k" else li.xt_v)) + 1.0
        assert (np.abs(xh.cpu().numpy() - oxh) / scale).max() < 2e-4
        assert np.abs(ret[:, col].cpu().numpy() - oR).max() < 2e-4
    # only some outputs requested
    only = torch.zeros(n_tok, 2, device="cuda")
    B.twkv_gate_soft(gc.h, 0, xk, xv, retain=only)
    torch.testing.assert_close(only, ret, rtol=0, atol=0)
    gc.close()
