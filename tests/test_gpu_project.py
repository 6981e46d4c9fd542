"""GPU parity of the spectral projection (Eq. 1) through the C ABI against the fp64 oracle.

Bar: the library accumulates the exact 16-bit products in fp32 and rounds once to the 16-bit type, so each
output must lie within half a unit in the last place of the 16-bit type around the exact value, widened by
the fp32 accumulation error (at most d_kv roundings of 2^-24 relative to sum_j |x_j U_jn|).  Most outputs then
carry exactly the bits of the oracle's rounding of the exact value; one whose exact value lies within the
accumulation error of a rounding boundary may land on the neighbouring 16-bit value (about sqrt(d_kv) 2^-24 /
2^-11 = 0.4 % of the outputs per unit of cancellation sum|x_j U_jn| / |x~_n|), so the share of identical bits is
only required to exceed 98 %.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_04411_b200 import workloads
from tests.helpers import bits16, dtype_name

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding
    return binding


def make_inputs(seed, n_tok, d, dtype, n_outliers=8):
    ch = workloads.outlier_channels(seed, d, n_outliers)
    ck, cv = workloads.raw_states(seed + 1, 4096, d, k_outliers=ch)
    U_k = workloads.pca_basis(ck).to(dtype)
    U_v = workloads.pca_basis(cv).to(dtype)
    xk, xv = workloads.raw_states(seed + 2, n_tok, d, k_outliers=ch)
    return xk.to(dtype), xv.to(dtype), U_k, U_v


def check_side(got_bits, x, U, dtype, rows=None):
    dn = dtype_name(dtype)
    xw = oracle.widen16(bits16(x), dn)
    Uw = oracle.widen16(bits16(U), dn)
    if rows is not None:
        xw = xw[rows]
        got_bits = got_bits[rows]
    exact = oracle.project(xw, Uw)
    want_bits = oracle.narrow16(exact, dn)
    got = oracle.widen16(got_bits, dn)
    eps = 2.0 ** (-11 if dn == "f16" else -8)
    half_ulp = np.maximum(np.abs(exact) * eps, 2.0 ** -25)              # fp16 subnormal spacing 2^-24
    acc = (np.abs(xw) @ np.abs(Uw)) * (x.shape[1] * 2.0 ** -24)
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - exact) <= half_ulp + acc), float(np.max(np.abs(got - exact) - half_ulp - acc))
    same = float(np.mean(got_bits == want_bits))
    assert same >= 0.98, same
    return same


def run(B, seed, n_tok, d, dtype, sides=(True, True)):
    xk, xv, U_k, U_v = make_inputs(seed, n_tok, d, dtype)
    xk_g, xv_g, Uk_g, Uv_g = (t.cuda().contiguous() for t in (xk, xv, U_k, U_v))
    ws = torch.empty(B.twkv_projector_required_bytes(d), dtype=torch.uint8, device="cuda")
    pj = B.twkv_projector_create(Uk_g if sides[0] else None, Uv_g if sides[1] else None, ws)
    sentinel = 0x7E01 if dtype == torch.float16 else 0x7FC1                # a NaN pattern: every element must be overwritten
    ok_ = torch.full((n_tok + 3, d), sentinel, dtype=torch.int16, device="cuda").view(dtype)
    ov_ = torch.full((n_tok + 3, d), sentinel, dtype=torch.int16, device="cuda").view(dtype)
    B.twkv_project(pj, xk_g if sides[0] else None, xv_g if sides[1] else None,
                   ok_ if sides[0] else None, ov_ if sides[1] else None, n_tok=n_tok)
    assert B.twkv_projector_status(pj) == B.TWKV_OK
    B.twkv_projector_destroy(pj)
    for on, out, x, U in ((sides[0], ok_, xk, U_k), (sides[1], ov_, xv, U_v)):
        bits = bits16(out.cpu())
        if on:
            check_side(bits[:n_tok], x, U, dtype)
        else:
            assert np.all(bits[:n_tok] == sentinel)
        assert np.all(bits[n_tok:] == sentinel)                            # rows past the last token are left alone


def test_project_fp16_ragged_two_sides(B):
    run(B, 31, 1000, 1024, torch.float16)


def test_project_pairs_fp16_ragged_last_pair_half_empty(B):
    # 1300 = 5 x 256 + 20: the last CTA pair has 20 valid rows in its first tile and none in its second
    run(B, 37, 1300, 1024, torch.float16)


def test_project_pairs_bf16_two_slabs_value_side_only(B):
    run(B, 38, 1024 + 129, 512, torch.bfloat16, sides=(False, True))


def test_project_bf16_two_slabs(B):
    run(B, 32, 300, 512, torch.bfloat16)


def test_project_three_narrow_slabs_value_side_only(B):
    run(B, 33, 129, 384, torch.float16, sides=(False, True))


def test_project_key_side_only_single_token_and_empty(B):
    run(B, 34, 1, 1024, torch.float16, sides=(True, False))
    d = 256
    _, _, U_k, U_v = make_inputs(35, 4, d, torch.float16)
    ws = torch.empty(B.twkv_projector_required_bytes(d), dtype=torch.uint8, device="cuda")
    pj = B.twkv_projector_create(U_k.cuda(), None, ws)
    x = torch.zeros(4, d, dtype=torch.float16, device="cuda")
    out = torch.ones(4, d, dtype=torch.float16, device="cuda")
    B.twkv_project(pj, x, None, out, None, n_tok=0)                        # nothing to do, nothing written
    assert bool((out == 1).all())
    with pytest.raises(B.TwkvError) as e:                                  # value side has no basis
        B.twkv_project(pj, None, x, None, out)
    assert e.value.code == B.TWKV_ERR_INVALID_ARG
    with pytest.raises(B.TwkvError) as e:                                  # in place is refused
        B.twkv_project(pj, x, None, x, None)
    assert e.value.code == B.TWKV_ERR_INVALID_ARG
    assert B.twkv_projector_status(pj) == B.TWKV_OK
    B.twkv_projector_destroy(pj)


def test_project_benchmark_size_sampled_rows(B):
    # the launch bench.py times (524 288 tokens, both sides, CTA-pair kernel), checked on sampled rows: the first and last
    # tile, tile and pair boundaries, and a seeded random draw
    n, d, dtype = 16 * 32768, 1024, torch.float16
    ch = workloads.outlier_channels(51, d, 8)
    ck, cv = workloads.raw_states(52, 4096, d, k_outliers=ch)
    U_k, U_v = workloads.pca_basis(ck).to(dtype), workloads.pca_basis(cv).to(dtype)
    xk, xv = workloads.raw_states(53, n, d, device="cuda", k_outliers=ch)
    xk, xv = xk.to(dtype), xv.to(dtype)
    ws = torch.empty(B.twkv_projector_required_bytes(d), dtype=torch.uint8, device="cuda")
    pj = B.twkv_projector_create(U_k.cuda(), U_v.cuda(), ws)
    ok_, ov_ = torch.empty_like(xk), torch.empty_like(xv)
    B.twkv_project(pj, xk, xv, ok_, ov_)
    assert B.twkv_projector_status(pj) == B.TWKV_OK
    B.twkv_projector_destroy(pj)
    rng = np.random.default_rng(54)
    rows = np.unique(np.concatenate([np.arange(0, 130), np.arange(255, 258), np.arange(n - 130, n), rng.integers(0, n, 256)]))
    idx = torch.from_numpy(rows).cuda()
    for out, x, U in ((ok_, xk, U_k), (ov_, xv, U_v)):
        check_side(bits16(out[idx].cpu()), x[idx].cpu(), U, dtype)


def test_project_identity_and_permutation_are_exact(B):
    d, n = 1024, 260
    g = torch.Generator().manual_seed(36)
    x = torch.randn(n, d, generator=g).to(torch.float16)
    P = torch.zeros(d, d, dtype=torch.float16)
    P[torch.arange(d), (torch.arange(d) + 1) % d] = 1.0                    # spectral axis j + 1 <- input dimension j
    ws = torch.empty(B.twkv_projector_required_bytes(d), dtype=torch.uint8, device="cuda")
    pj = B.twkv_projector_create(torch.eye(d, dtype=torch.float16).cuda(), P.cuda(), ws)
    a = torch.empty(n, d, dtype=torch.float16, device="cuda")
    b = torch.empty(n, d, dtype=torch.float16, device="cuda")
    B.twkv_project(pj, x.cuda(), x.cuda(), a, b)
    assert B.twkv_projector_status(pj) == B.TWKV_OK
    B.twkv_projector_destroy(pj)
    assert torch.equal(a.cpu(), x)
    assert torch.equal(b.cpu(), torch.roll(x, 1, dims=1))


def test_project_then_compress_and_decode_from_raw_states(B):
    """Raw states -> Eq. 1 on the device -> compress -> decode, against the oracle taking the same steps."""
    from tests.helpers import GpuCache, attn_errors
    dtype, d, n_seq, ctx, Hq = torch.float16, 1024, 2, 700, 32
    li = workloads.build_layer(41, n_seq=n_seq, ctx=ctx, n_q_heads=Hq, dtype=dtype, device="cpu", mode="forced", keep_raw=True)
    n_tok = n_seq * ctx
    xk, xv = li.raw_k.to(dtype), li.raw_v.to(dtype)
    U_k, U_v = li.U_k.to(dtype), li.U_v.to(dtype)
    ws = torch.empty(B.twkv_projector_required_bytes(d), dtype=torch.uint8, device="cuda")
    pj = B.twkv_projector_create(U_k.cuda(), U_v.cuda(), ws)
    xt_k = torch.empty(n_tok, d, dtype=dtype, device="cuda")
    xt_v = torch.empty(n_tok, d, dtype=dtype, device="cuda")
    B.twkv_project(pj, xk.cuda(), xv.cuda(), xt_k, xt_v)
    assert B.twkv_projector_status(pj) == B.TWKV_OK
    B.twkv_projector_destroy(pj)
    ranks = li.ranks.numpy()
    gc = GpuCache(B, n_layers=1, n_q_heads=Hq, n_kv_heads=8, dtype=dtype, out_dtype=torch.float32, max_seqs=n_seq,
                  max_tokens_per_seq=ctx, payload_bytes=int((-(-ranks.astype(np.int64) // 64) * 128).sum()))
    B.twkv_cache_set_layer_params(gc.h, 0, li.Uinv_k.cuda(), li.Uinv_v.cuda())
    lv = torch.from_numpy(np.ascontiguousarray(ranks.astype(np.int16))).cuda()
    B.twkv_compress(gc.h, 0, xt_k, xt_v, li.seq_ids.cuda(), li.positions.cuda(), None, lv, B.TWKV_GATE_FORCED)
    out = torch.empty(n_seq, Hq, 128, dtype=torch.float32, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q.cuda(), torch.arange(n_seq, dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    gc.close()
    # oracle: the same chain in fp64 with the one 16-bit rounding after Eq. 1
    dn = "f16"
    w = lambda t: oracle.widen16(bits16(t), dn)
    ok_ = oracle.widen16(oracle.narrow16(oracle.project(w(xk), w(U_k)), dn), dn)
    ov_ = oracle.widen16(oracle.narrow16(oracle.project(w(xv), w(U_v)), dn), dn)
    pos = li.positions.numpy()
    for s in range(n_seq):
        sl = slice(s * ctx, (s + 1) * ctx)
        want = oracle.decode_attn(ok_[sl], ov_[sl], ranks[sl, 0], ranks[sl, 1], pos[sl], w(li.Uinv_k), w(li.Uinv_v),
                                  w(li.q[s]), 8, 500000.0, 128 ** -0.5)
        max_abs, rel = attn_errors(out[s].cpu().numpy(), want)
        assert max_abs <= 2e-3 and rel <= 1e-3, (s, max_abs, rel)
