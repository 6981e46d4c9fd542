"""Pins for the fp64 oracle: closed forms, invariants, special cases, brute force.

None of these re-type the oracle's own formula; each checks it against a value
the paper or the mathematics fixes, so that a dropped term, wrong sign, wrong
index or transposed operand in the oracle fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

import oracle
from oracle.cache_image import CacheImage, PANEL, TILE

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append([float(v) for v in line.split()])
    return rows


# ----------------------------------------------------------------------------- gate
def test_gate_uniform_logits_closed_form():
    # p_j = 1/d, c_n = n/d (exact for d a power of two); r = d - #{n : n/d <= tau}
    for d, tau, want in _golden("gate_closed_forms.txt"):
        d = int(d)
        r, _ = oracle.gate_rank(np.zeros((1, d)), tau)
        assert int(r[0]) == int(want), (d, tau)


def test_gate_strictness_at_equality():
    # tau d integer: c_{tau d} == tau exactly, Eq. 8 is strict so that entry is discarded
    d = 1024
    r_eq, margin = oracle.gate_rank(np.zeros((1, d)), 0.125)
    assert r_eq[0] == d - 128 and margin[0] == 0.0
    r_below, _ = oracle.gate_rank(np.zeros((1, d)), np.nextafter(0.125, 0.0))
    assert r_below[0] == d - 127


@pytest.mark.parametrize("d", [8, 64, 1024])
def test_gate_one_hot_pins_flip_direction(d):
    # all mass on truncation index k (1-based): c_n = 1[n >= k]; m_i = c_{d+1-i} = 1[i <= d+1-k]
    for k in [1, 2, d // 2, d - 1, d]:
        z = np.full((1, d), -800.0)
        z[0, k - 1] = 0.0
        r, margin, m = oracle.gate_rank(z, 0.1, want_soft=True)
        assert r[0] == d - k + 1
        want = (np.arange(1, d + 1) <= d + 1 - k).astype(float)
        np.testing.assert_array_equal(m[0], want)
        assert margin[0] > 0.99


def test_gate_invariants():
    rng = np.random.default_rng(0)
    d = 256
    z = rng.normal(size=(64, d)) * 3
    r, margin, m = oracle.gate_rank(z, 0.1, want_soft=True)
    assert np.all(np.diff(m, axis=1) <= 0)                 # soft mask non-increasing
    np.testing.assert_allclose(m[:, 0], 1.0, atol=1e-12)    # m_1 = total probability
    assert np.all((r >= 1) & (r <= d))
    hard = m > 0.1
    for t in range(len(r)):                                # hard mask is a prefix of ones
        assert hard[t, :r[t]].all() and not hard[t, r[t]:].any()
    # mean of the soft mask: sum_i m_i = sum_n (d + 1 - n) ... = sum_j p_j (d + 1 - j): check via p
    p = np.exp(z - z.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    np.testing.assert_allclose(m.sum(1), (p * (d - np.arange(d))).sum(1), rtol=1e-12)
    # r non-increasing in tau; constant logit shift changes nothing
    prev = None
    for tau in [0.01, 0.05, 0.1, 0.3, 0.7, 0.99]:
        rt, _ = oracle.gate_rank(z, tau)
        if prev is not None:
            assert np.all(rt <= prev)
        prev = rt
    r2, _ = oracle.gate_rank(z + 123.25, 0.1)
    np.testing.assert_array_equal(r, r2)


def test_gate_two_point_distribution():
    # logits with mass a on index k1 and 1-a on k2 > k1: r = d-k1+1 if a > tau else d-k2+1
    d = 128
    for a in [0.05, 0.2]:
        z = np.full((1, d), -800.0)
        z[0, 9] = math.log(a)
        z[0, 99] = math.log(1 - a)
        r, _ = oracle.gate_rank(z, 0.1)
        assert r[0] == (d - 10 + 1 if a > 0.1 else d - 100 + 1)


def test_gate_logits_orientation_and_bias():
    d = 16
    rng = np.random.default_rng(1)
    x = rng.normal(size=(3, d))
    b = rng.normal(size=d)
    np.testing.assert_allclose(oracle.gate_logits(x, np.eye(d), b), x + b, rtol=0, atol=1e-15)
    # a single non-zero weight W[j, n] routes input component j to logit n (not n to j)
    W = np.zeros((d, d)); W[2, 5] = 3.0
    z = oracle.gate_logits(x, W, None)
    want = np.zeros_like(x); want[:, 5] = 3.0 * x[:, 2]
    np.testing.assert_allclose(z, want, atol=1e-15)
    # linearity
    W = rng.normal(size=(d, d))
    z1 = oracle.gate_logits(x, W, b); z2 = oracle.gate_logits(2 * x, W, b)
    np.testing.assert_allclose(z2 - z1, z1 - b, rtol=1e-12, atol=1e-12)


def _rand_orth(rng, d):
    q, _ = np.linalg.qr(rng.normal(size=(d, d)))
    return q


# ------------------------------------------------------------------ spectral projection
def test_project_closed_forms_pin_orientation():
    rng = np.random.default_rng(21)
    d = 24
    x = rng.normal(size=(6, d))
    # cyclic shift: U[j, (j + 1) % d] = 1 sends input dimension j to spectral axis j + 1 (x U, not x U^T)
    P = np.zeros((d, d))
    P[np.arange(d), (np.arange(d) + 1) % d] = 1.0
    np.testing.assert_array_equal(oracle.project(x, P), np.roll(x, 1, axis=1))
    # diagonal U scales axis n by s_n; identity leaves x alone
    s_ = rng.normal(size=d)
    np.testing.assert_array_equal(oracle.project(x, np.diag(s_)), x * s_[None, :])
    np.testing.assert_array_equal(oracle.project(x, np.eye(d)), x)
    # rank one U = a b^T: x~ = (x . a) b
    a, b = rng.normal(size=d), rng.normal(size=d)
    np.testing.assert_allclose(oracle.project(x, np.outer(a, b)), (x @ a)[:, None] * b[None, :], rtol=1e-12, atol=1e-12)
    # one-hot input row j reads out row j of U
    M = np.arange(d * d, dtype=np.float64).reshape(d, d)
    np.testing.assert_array_equal(oracle.project(np.eye(d)[3:4], M)[0], M[3])


def test_project_then_full_rank_reconstruct_is_identity_and_preserves_energy():
    rng = np.random.default_rng(22)
    d = 64
    x = rng.normal(size=(9, d))
    U = _rand_orth(rng, d)
    xt = oracle.project(x, U)
    np.testing.assert_allclose((xt ** 2).sum(1), (x ** 2).sum(1), rtol=1e-12)          # orthogonal U: Parseval
    np.testing.assert_allclose(oracle.reconstruct(xt, np.full(9, d, np.int32), U.T), x, atol=1e-12)   # Eq. 3 undoes Eq. 1
    G = rng.normal(size=(d, d)) + 5 * np.eye(d)                                        # learnable U need not stay orthogonal
    np.testing.assert_allclose(oracle.reconstruct(oracle.project(x, G), np.full(9, d, np.int32), np.linalg.inv(G)), x, atol=1e-10)


def test_project_with_pca_eigenvectors_orders_the_energy():
    # U = eigenvectors of the calibration covariance, largest eigenvalue first: the projected dimensions are
    # uncorrelated and their variances are the eigenvalues in descending order (what lets Eq. 2 prune the tail)
    rng = np.random.default_rng(23)
    d = 40
    A = rng.normal(size=(d, d)) * (0.85 ** np.arange(d))[None, :]
    x = rng.normal(size=(3000, d)) @ A.T
    x = x - x.mean(0)
    lam, vec = np.linalg.eigh(np.cov(x.T))
    order = np.argsort(lam)[::-1]
    U = vec[:, order]
    C = np.cov(oracle.project(x, U).T)
    np.testing.assert_allclose(np.diag(C), lam[order], rtol=1e-9)
    assert np.all(np.diff(np.diag(C)) <= 1e-12)
    off = C - np.diag(np.diag(C))
    assert np.abs(off).max() < 1e-10 * lam.max()


def test_narrow16_round_to_nearest_even():
    # fp16: 11 significand bits; bf16: 8.  Halfway cases go to the even neighbour, everything else to the nearest.
    f16 = oracle.narrow16(np.array([1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -30, -2.5, 65504.0, 65520.0, 0.0]), "f16")
    np.testing.assert_array_equal(f16, np.array([0x3C00, 0x3C00, 0x3C02, 0x3C01, 0xC100, 0x7BFF, 0x7C00, 0x0000], dtype=np.uint16))
    b16 = oracle.narrow16(np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40, -2.5, 3.0e38, 0.0,
                                    1.0 + 2.0 ** -8 - 2.0 ** -40]), "bf16")
    np.testing.assert_array_equal(b16, np.array([0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xC020, 0x7F62, 0x0000, 0x3F80], dtype=np.uint16))
    # widening what was narrowed is exact, and narrowing representable values changes nothing
    rng = np.random.default_rng(24)
    for dt in ("f16", "bf16"):
        bits = oracle.narrow16(rng.normal(size=1000) * 8, dt)
        np.testing.assert_array_equal(oracle.narrow16(oracle.widen16(bits, dt), dt), bits)
        v = rng.normal(size=1000) * 8
        err = np.abs(oracle.widen16(oracle.narrow16(v, dt), dt) - v)
        assert np.all(err <= np.abs(v) * 2.0 ** (-11 if dt == "f16" else -8))


# ---------------------------------------------------------------- truncate / reconstruct
def test_reconstruct_parseval_tail_energy():
    rng = np.random.default_rng(2)
    d = 64
    U = _rand_orth(rng, d)
    x = rng.normal(size=(10, d))
    xt = x @ U                                              # Eq. 1
    for rr in [1, 7, 32, 63, 64]:
        r = np.full(10, rr, dtype=np.int32)
        xbar = oracle.reconstruct(xt, r, U.T)
        tail = (xt[:, rr:] ** 2).sum(1)
        np.testing.assert_allclose(((x - xbar) ** 2).sum(1), tail, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(oracle.reconstruct(xt, np.full(10, d, np.int32), U.T), x, atol=1e-12)


def test_reconstruct_non_orthogonal_full_rank_and_row_selection():
    rng = np.random.default_rng(3)
    d = 32
    U = rng.normal(size=(d, d)) + 4 * np.eye(d)
    Uinv = np.linalg.inv(U)
    x = rng.normal(size=(5, d))
    np.testing.assert_allclose(oracle.reconstruct(x @ U, np.full(5, d, np.int32), Uinv), x, atol=1e-10)
    # rank 1 keeps spectral component 0 only: xbar = x~_0 * (row 0 of Uinv), not column 0
    xt = x @ U
    xbar = oracle.reconstruct(xt, np.ones(5, np.int32), Uinv)
    np.testing.assert_allclose(xbar, xt[:, :1] * Uinv[0:1, :], atol=1e-12)
    # per-token ranks are honoured independently
    r = np.array([1, 5, 9, 32, 17], dtype=np.int32)
    xbar = oracle.reconstruct(xt, r, Uinv)
    for t in range(5):
        np.testing.assert_allclose(xbar[t], xt[t, :r[t]] @ Uinv[:r[t]], atol=1e-12)
    # entries past r never influence the result (they were physically discarded, Eq. 2)
    junk = xt.copy()
    for t in range(5):
        junk[t, r[t]:] = 1e30
    np.testing.assert_array_equal(oracle.reconstruct(junk, r, Uinv), xbar)
    np.testing.assert_array_equal(oracle.truncate(xt, r)[1, 5:], 0.0)


def test_pca_basis_is_optimal_on_its_calibration_set():
    import torch
    from paper_2603_04411_b200 import workloads
    rng = np.random.default_rng(4)
    d = 48
    A = rng.normal(size=(d, d)) * (0.9 ** np.arange(d))[None, :]
    x = rng.normal(size=(4000, d)) @ A.T
    x = x - x.mean(0)
    U = workloads.pca_basis(torch.from_numpy(x)).numpy()
    lam = np.sort(np.linalg.eigvalsh(np.cov(x.T)))[::-1]
    R = _rand_orth(rng, d)
    for rr in [4, 12, 24]:
        r = np.full(len(x), rr, np.int32)
        mse = ((x - oracle.reconstruct(x @ U, r, U.T)) ** 2).sum(1).mean()
        np.testing.assert_allclose(mse * len(x) / (len(x) - 1), lam[rr:].sum(), rtol=1e-8)
        mse_rand = ((x - oracle.reconstruct(x @ R, r, R.T)) ** 2).sum(1).mean()
        assert mse <= mse_rand


# ----------------------------------------------------------------------------- RoPE
def _rope_complex(k, pos, H, dh, base):
    """Independent RoPE: treat (k_i, k_{i+dh/2}) as a complex number and multiply by e^{i pos theta_i}."""
    k = k.reshape(len(pos), H, dh)
    half = dh // 2
    zc = k[..., :half] + 1j * k[..., half:]
    theta = base ** (-2.0 * np.arange(half) / dh)
    zc = zc * np.exp(1j * np.asarray(pos, dtype=np.float64)[:, None, None] * theta[None, None, :])
    return np.concatenate([zc.real, zc.imag], axis=-1).reshape(len(pos), H * dh)


def test_rope_pins():
    rng = np.random.default_rng(5)
    H, dh, base = 3, 16, 10000.0
    k = rng.normal(size=(6, H * dh))
    pos = np.array([0, 1, 2, 77, 4095, 131071], dtype=np.int32)
    kr = oracle.rope(k, pos, H, dh, base)
    np.testing.assert_array_equal(kr[0], k[0])                                  # position 0 = identity
    np.testing.assert_allclose(kr, _rope_complex(k, pos, H, dh, base), atol=1e-9)
    # pair norms preserved
    a = k.reshape(6, H, 2, dh // 2); b = kr.reshape(6, H, 2, dh // 2)
    np.testing.assert_allclose((a ** 2).sum(2), (b ** 2).sum(2), rtol=1e-12)
    # textbook value: pair (1, 0) at position p, frequency 0 (theta = 1) -> (cos p, sin p)
    e = np.zeros((1, dh)); e[0, 0] = 1.0
    out = oracle.rope(e, np.array([3], np.int32), 1, dh, base)
    np.testing.assert_allclose([out[0, 0], out[0, dh // 2]], [math.cos(3.0), math.sin(3.0)], atol=1e-15)
    # last frequency: theta = base^(-(dh-2)/dh)
    e = np.zeros((1, dh)); e[0, dh // 2 - 1] = 1.0
    out = oracle.rope(e, np.array([1000], np.int32), 1, dh, base)
    th = base ** (-(dh - 2) / dh)
    np.testing.assert_allclose([out[0, dh // 2 - 1], out[0, dh - 1]], [math.cos(1000 * th), math.sin(1000 * th)], atol=1e-13)


# ------------------------------------------------------------------------ attention
def _exact_attention_from_raw(x_k, x_v, pos, q, Hkv, base, scale):
    """Attention straight from the raw states x: never touches U or the oracle's reconstruct."""
    Hq, dh = q.shape
    kr = _rope_complex(x_k, pos, Hkv, dh, base).reshape(len(pos), Hkv, dh)
    v = x_v.reshape(len(pos), Hkv, dh)
    out = np.zeros((Hq, dh))
    for h in range(Hq):
        g = h // (Hq // Hkv)
        s = kr[:, g, :] @ q[h] * scale
        a = np.exp(s - s.max()); a /= a.sum()
        out[h] = a @ v[:, g, :]
    return out


def test_uncompressed_level_equals_exact_attention():
    rng = np.random.default_rng(6)
    Hkv, Hq, dh, T = 2, 4, 16, 37
    d = Hkv * dh
    Uk, Uv = _rand_orth(rng, d), _rand_orth(rng, d)
    xk, xv = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    q = rng.normal(size=(Hq, dh))
    pos = rng.permutation(200)[:T].astype(np.int32)
    full = np.full(T, d, np.int32)
    out = oracle.decode_attn(xk @ Uk, xv @ Uv, full, full, pos, Uk.T, Uv.T, q, Hkv, 10000.0, dh ** -0.5)
    want = _exact_attention_from_raw(xk, xv, pos, q, Hkv, 10000.0, dh ** -0.5)
    np.testing.assert_allclose(out, want, atol=1e-11)


def test_bruteforce_tiny_with_truncation():
    # literal double sums in Python on T <= 8, Hkv = 2, dh = 4, d_kv = 8, mixed ranks, non-orthogonal U
    rng = np.random.default_rng(7)
    Hkv, Hq, dh, T = 2, 4, 4, 7
    d = Hkv * dh
    Uik, Uiv = rng.normal(size=(d, d)), rng.normal(size=(d, d))
    xk, xv = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    rk = rng.integers(1, d + 1, T).astype(np.int32)
    rv = rng.integers(1, d + 1, T).astype(np.int32)
    pos = np.arange(T, dtype=np.int32) * 3
    q = rng.normal(size=(Hq, dh))
    base, scale = 100.0, 0.5
    out = oracle.decode_attn(xk, xv, rk, rv, pos, Uik, Uiv, q, Hkv, base, scale)
    for h in range(Hq):
        g = h // 2
        s = []
        vb = []
        for t in range(T):
            kbar = [sum(xk[t][j] * Uik[j][n] for j in range(rk[t])) for n in range(d)]
            vbar = [sum(xv[t][j] * Uiv[j][n] for j in range(rv[t])) for n in range(d)]
            kh = kbar[g * dh:(g + 1) * dh]
            rot = list(kh)
            for i in range(dh // 2):
                ang = pos[t] * base ** (-2.0 * i / dh)
                rot[i] = kh[i] * math.cos(ang) - kh[i + dh // 2] * math.sin(ang)
                rot[i + dh // 2] = kh[i + dh // 2] * math.cos(ang) + kh[i] * math.sin(ang)
            s.append(sum(q[h][i] * rot[i] for i in range(dh)) * scale)
            vb.append(vbar[g * dh:(g + 1) * dh])
        mx = max(s)
        e = [math.exp(v - mx) for v in s]
        for i in range(dh):
            want = sum(e[t] * vb[t][i] for t in range(T)) / sum(e)
            assert abs(out[h][i] - want) < 1e-12


def _mk_case(rng, T=50, Hkv=2, Hq=4, dh=8):
    d = Hkv * dh
    return dict(xk=rng.normal(size=(T, d)), xv=rng.normal(size=(T, d)),
                rk=rng.integers(1, d + 1, T).astype(np.int32), rv=rng.integers(1, d + 1, T).astype(np.int32),
                pos=rng.permutation(1000)[:T].astype(np.int32),
                Uk=rng.normal(size=(d, d)), Uv=rng.normal(size=(d, d)),
                q=rng.normal(size=(Hq, dh)), Hkv=Hkv, dh=dh)


def _run(c, idx=None, q=None, pos=None):
    idx = slice(None) if idx is None else idx
    return oracle.decode_attn(c["xk"][idx], c["xv"][idx], c["rk"][idx], c["rv"][idx],
                              (c["pos"] if pos is None else pos)[idx], c["Uk"], c["Uv"],
                              c["q"] if q is None else q, c["Hkv"], 10000.0, c["dh"] ** -0.5)


def test_attention_permutation_and_single_token():
    rng = np.random.default_rng(8)
    c = _mk_case(rng)
    out = _run(c)
    perm = rng.permutation(len(c["pos"]))
    np.testing.assert_allclose(_run(c, perm), out, atol=1e-12)       # positions travel with tokens
    one = _run(c, slice(3, 4))
    vbar = oracle.reconstruct(c["xv"][3:4], c["rv"][3:4], c["Uv"]).reshape(c["Hkv"], c["dh"])
    for h in range(4):
        np.testing.assert_allclose(one[h], vbar[h // 2], atol=1e-13)  # T = 1: out = vbar whatever q is


def test_rope_common_shift_leaves_attention_unchanged():
    rng = np.random.default_rng(9)
    c = _mk_case(rng)
    out = _run(c)
    shift = 321
    q_rot = oracle.rope(c["q"].reshape(1, -1).repeat(1, 0), np.array([shift], np.int32), 4, c["dh"], 10000.0)
    np.testing.assert_allclose(_run(c, q=q_rot.reshape(4, c["dh"]), pos=c["pos"] + shift), out, atol=1e-10)


def test_split_lse_merge_and_absorbed_v_identities():
    """The GPU route (token splits merged by log-sum-exp; V accumulated in spectral space and
    projected once) is licensed by these identities of the plain definition."""
    rng = np.random.default_rng(10)
    c = _mk_case(rng, T=60)
    out = _run(c)
    Hkv, dh = c["Hkv"], c["dh"]
    d = Hkv * dh
    kbar = oracle.rope(oracle.reconstruct(c["xk"], c["rk"], c["Uk"]), c["pos"], Hkv, dh, 10000.0).reshape(-1, Hkv, dh)
    xhat_v = oracle.truncate(c["xv"], c["rv"])
    for h in range(4):
        g = h // 2
        s = kbar[:, g, :] @ c["q"][h] * dh ** -0.5
        parts = []
        for idx in (slice(0, 13), slice(13, 14), slice(14, 60)):
            mx = s[idx].max(); e = np.exp(s[idx] - mx)
            parts.append((mx, e.sum(), e @ xhat_v[idx]))                 # spectral-space accumulator [d]
        M = max(p[0] for p in parts)
        L = sum(p[1] * math.exp(p[0] - M) for p in parts)
        acc = sum(p[2] * math.exp(p[0] - M) for p in parts)
        merged = (acc / L) @ c["Uv"][:, g * dh:(g + 1) * dh]             # one projection at the end
        np.testing.assert_allclose(merged, out[h], atol=1e-11)


def test_truncation_changes_the_answer_by_the_dropped_terms():
    # guards against an oracle that ignores ranks: rank d vs rank d-1 must differ exactly by the last term
    rng = np.random.default_rng(11)
    c = _mk_case(rng, T=1)
    d = c["Hkv"] * c["dh"]
    c["rv"][:] = d
    full = _run(c)
    c["rv"][:] = d - 1
    cut = _run(c)
    diff = (full - cut).reshape(-1)
    want = c["xv"][0, d - 1] * c["Uv"][d - 1]
    np.testing.assert_allclose(diff, np.concatenate([want[:c["dh"]]] * 2 + [want[c["dh"]:]] * 2), atol=1e-12)


# ------------------------------------------------------------------- retain rate, image
def test_retain_rate_and_stored_bytes():
    rng = np.random.default_rng(12)
    d, S, n = 256, 3, 700
    ranks = rng.integers(1, d + 1, size=(n, 2)).astype(np.int32)
    assert abs(oracle.retain_rate(ranks[:, 0], d) - ranks[:, 0].mean() / d) < 1e-15
    assert oracle.retain_rate(np.full(5, d), d) == 1.0
    img = CacheImage(1, d, S, 1024, 4096)
    xk = rng.integers(1, 2 ** 16, size=(n, d)).astype(np.uint16)
    xv = rng.integers(1, 2 ** 16, size=(n, d)).astype(np.uint16)
    seq = rng.integers(0, S, n).astype(np.int32)
    pos = np.arange(n, dtype=np.int32)
    assert img.append(0, xk, xv, seq, pos, ranks)
    cls = -(-ranks // PANEL)
    assert img.stored_bytes() == int((cls * PANEL * 2).sum())
    # every token's row can be found again, in arrival order, zero-filled past r
    for side, x in ((0, xk), (1, xv)):
        seen = {}
        for i in range(n):
            k = img.key(side, int(seq[i]), int(cls[i, side]))
            g = seen.get(k, 0); seen[k] = g + 1
            tid = img.key_tiles[0][k][g // TILE]; slot = g % TILE
            s_, c_, nv, base = img.tile_desc[0, side, tid]
            assert s_ == seq[i] and c_ == cls[i, side] and slot < nv
            row = np.concatenate([img.blocks[base + j, slot * PANEL:(slot + 1) * PANEL] for j in range(c_)])
            r = ranks[i, side]
            np.testing.assert_array_equal(row[:r], x[i, :r])
            assert not row[r:].any()
            assert img.tile_rank[0, side, tid, slot] == r
            if side == 0:
                assert img.tile_aux[0, 0, tid, slot] == pos[i]
            else:
                link = img.tile_aux[0, 1, tid, slot]
                assert img.tile_aux[0, 0, link // TILE, link % TILE] == pos[i]   # link finds the same token's K row
    # blocks of distinct tiles never overlap
    used = []
    for side in range(2):
        for tid in range(int(img.n_tiles[0, side])):
            _, c_, _, base = img.tile_desc[0, side, tid]
            used += list(range(base, base + c_))
    assert len(used) == len(set(used)) == img.next_block


def test_image_append_in_two_calls_matches_one_call_logically():
    rng = np.random.default_rng(13)
    d, S, n = 128, 2, 300
    ranks = rng.integers(1, d + 1, size=(n, 2)).astype(np.int32)
    xk = rng.integers(0, 2 ** 16, size=(n, d)).astype(np.uint16)
    xv = rng.integers(0, 2 ** 16, size=(n, d)).astype(np.uint16)
    seq = rng.integers(0, S, n).astype(np.int32)
    pos = np.arange(n, dtype=np.int32)
    a = CacheImage(1, d, S, 512, 1024); a.append(0, xk, xv, seq, pos, ranks)
    b = CacheImage(1, d, S, 512, 1024)
    b.append(0, xk[:111], xv[:111], seq[:111], pos[:111], ranks[:111])
    b.append(0, xk[111:], xv[111:], seq[111:], pos[111:], ranks[111:])
    for k in range(2 * S * a.NC):
        ra = [a.blocks[a.tile_desc[0, k // (S * a.NC), t, 3]] for t in a.key_tiles[0][k]]
        rb = [b.blocks[b.tile_desc[0, k // (S * a.NC), t, 3]] for t in b.key_tiles[0][k]]
        assert len(ra) == len(rb)
        for x, y in zip(ra, rb):
            np.testing.assert_array_equal(x, y)


def test_image_capacity_refusal_leaves_state_unchanged():
    d = 128
    img = CacheImage(1, d, 1, 256, 3)
    x = np.ones((200, d), np.uint16)
    seq = np.zeros(200, np.int32); pos = np.arange(200, dtype=np.int32)
    ranks = np.full((200, 2), 128, np.int32)            # class 2: 2 tiles x 2 blocks x 2 sides = 8 blocks > 3
    assert not img.append(0, x, x, seq, pos, ranks)
    assert img.next_block == 0 and img.n_tiles.sum() == 0 and img.fill.sum() == 0


# ---------------------------------------------------------------------------------------------
# chunked-prefill attention: causal queries over the compressed cache
def test_prefill_one_query_seeing_everything_is_decode():
    rng = np.random.default_rng(21)
    Hkv, Hq, dh, T = 2, 4, 8, 19
    d = Hkv * dh
    Uik, Uiv = rng.normal(size=(d, d)), rng.normal(size=(d, d))
    xk, xv = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    rk = rng.integers(1, d + 1, T).astype(np.int32)
    rv = rng.integers(1, d + 1, T).astype(np.int32)
    pos = rng.permutation(50)[:T].astype(np.int32)
    q = rng.normal(size=(1, Hq, dh))
    got = oracle.prefill_attn(xk, xv, rk, rv, pos, Uik, Uiv, q, np.array([int(pos.max())]), Hkv, 1000.0, 0.3)
    want = oracle.decode_attn(xk, xv, rk, rv, pos, Uik, Uiv, q[0], Hkv, 1000.0, 0.3)
    np.testing.assert_allclose(got[0], want, rtol=0, atol=1e-13)


def test_prefill_bruteforce_tiny_causal():
    # literal Python sums with the causal mask written out, T = 7, mixed ranks, non-orthogonal U
    rng = np.random.default_rng(22)
    Hkv, Hq, dh, T = 2, 4, 4, 7
    d = Hkv * dh
    Uik, Uiv = rng.normal(size=(d, d)), rng.normal(size=(d, d))
    xk, xv = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    rk = rng.integers(1, d + 1, T).astype(np.int32)
    rv = rng.integers(1, d + 1, T).astype(np.int32)
    pos = np.array([0, 2, 3, 5, 8, 9, 12], dtype=np.int32)
    q_pos = np.array([3, 0, 12, 7])
    q = rng.normal(size=(len(q_pos), Hq, dh))
    base, scale = 50.0, 0.7
    got = oracle.prefill_attn(xk, xv, rk, rv, pos, Uik, Uiv, q, q_pos, Hkv, base, scale)
    for i, qp in enumerate(q_pos):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            num, den, smax, sc, vbars = [0.0] * dh, 0.0, -1e300, [], []
            for t in range(T):
                if pos[t] > qp:
                    continue                                     # causal: the query does not see later tokens
                kbar = [sum(xk[t][j] * Uik[j][g * dh + n] for j in range(rk[t])) for n in range(dh)]
                vbars.append([sum(xv[t][j] * Uiv[j][g * dh + n] for j in range(rv[t])) for n in range(dh)])
                rot = list(kbar)
                for a in range(dh // 2):
                    ang = pos[t] * base ** (-2.0 * a / dh)
                    rot[a] = kbar[a] * math.cos(ang) - kbar[a + dh // 2] * math.sin(ang)
                    rot[a + dh // 2] = kbar[a + dh // 2] * math.cos(ang) + kbar[a] * math.sin(ang)
                sc.append(scale * sum(q[i][h][n] * rot[n] for n in range(dh)))
            smax = max(sc)
            w = [math.exp(x - smax) for x in sc]
            den = sum(w)
            for n in range(dh):
                num[n] = sum(w[k] * vbars[k][n] for k in range(len(w))) / den
            np.testing.assert_allclose(got[i][h], num, rtol=0, atol=1e-12)


def test_prefill_full_rank_equals_exact_causal_attention_and_ignores_the_future():
    rng = np.random.default_rng(23)
    Hkv, Hq, dh, T = 2, 4, 16, 33
    d = Hkv * dh
    Uk, Uv = _rand_orth(rng, d), _rand_orth(rng, d)
    xk, xv = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    pos = np.arange(T, dtype=np.int32)
    full = np.full(T, d, np.int32)
    q_pos = np.array([0, 5, 17, 32])
    q = rng.normal(size=(len(q_pos), Hq, dh))
    got = oracle.prefill_attn(xk @ Uk, xv @ Uv, full, full, pos, Uk.T, Uv.T, q, q_pos, Hkv, 10000.0, dh ** -0.5)
    for i, qp in enumerate(q_pos):
        want = _exact_attention_from_raw(xk[:qp + 1], xv[:qp + 1], pos[:qp + 1], q[i], Hkv, 10000.0, dh ** -0.5)
        np.testing.assert_allclose(got[i], want, atol=1e-11)
    # tokens after a query's position do not matter: replace them and compare
    xk2, xv2 = xk.copy(), xv.copy()
    xk2[18:] = rng.normal(size=(T - 18, d)); xv2[18:] = rng.normal(size=(T - 18, d))
    got2 = oracle.prefill_attn(xk2 @ Uk, xv2 @ Uv, full, full, pos, Uk.T, Uv.T, q, q_pos, Hkv, 10000.0, dh ** -0.5)
    np.testing.assert_array_equal(got[:3], got2[:3])
    # a query before every cached token sees nothing
    none = oracle.prefill_attn(xk @ Uk, xv @ Uv, full, full, pos + 5, Uk.T, Uv.T, q[:1], np.array([2]), Hkv, 10000.0, dh ** -0.5)
    assert not none.any()


# ---------------------------------------------------------------------------------------------
# soft gating (Eq. 6, Eq. 7, the soft Retain Rate of Eq. 9)
def test_soft_gate_closed_forms():
    d = 16
    # uniform logits: p_j = 1/d, c_n = n/d, m_i = c_{d+1-i} = (d+1-i)/d, mean = (d+1)/(2d)
    z = np.zeros((1, d))
    x = np.arange(1.0, d + 1)[None, :]
    m, xh, R = oracle.soft_gate(x, z)
    np.testing.assert_allclose(m[0], (d - np.arange(d)) / d, atol=1e-15)
    np.testing.assert_allclose(xh[0], x[0] * (d - np.arange(d)) / d, atol=1e-13)
    assert abs(R[0] - (d + 1) / (2 * d)) < 1e-15
    # all mass on truncation index k (1-based): c_n = [n >= k], m_i = [i <= d+1-k]: keeps d+1-k leading components
    for k in (1, 5, 16):
        z = np.full((1, d), -800.0); z[0, k - 1] = 0.0
        m, xh, R = oracle.soft_gate(x, z)
        want = (np.arange(1, d + 1) <= d + 1 - k).astype(float)
        np.testing.assert_array_equal(m[0], want)
        np.testing.assert_array_equal(xh[0], x[0] * want)
        assert R[0] == (d + 1 - k) / d
    # two-point mass: p_a = 0.25, p_b = 0.75 (a < b): m = 1 up to d+1-b, 0.25 up to d+1-a, 0 after
    a, b = 3, 11
    z = np.full((1, d), -800.0); z[0, a - 1] = math.log(0.25); z[0, b - 1] = math.log(0.75)
    m, _, R = oracle.soft_gate(x, z)
    idx = np.arange(1, d + 1)
    want = np.where(idx <= d + 1 - b, 1.0, np.where(idx <= d + 1 - a, 0.25, 0.0))
    np.testing.assert_allclose(m[0], want, atol=1e-15)
    assert abs(R[0] - want.mean()) < 1e-15


def test_soft_gate_invariants_and_link_to_hard_mask():
    rng = np.random.default_rng(31)
    n, d = 40, 64
    z = rng.normal(size=(n, d)) * 3
    x = rng.normal(size=(n, d))
    m, xh, R = oracle.soft_gate(x, z)
    assert np.all(np.diff(m, axis=1) <= 1e-15) and np.allclose(m[:, 0], 1.0) and np.all(m >= 0)
    np.testing.assert_allclose(xh, x * m, atol=0)
    # the hard mask of Eq. 8 is the soft mask thresholded: r = #{i : m_i > tau}
    for tau in (0.05, 0.1, 0.5):
        r, _ = oracle.gate_rank(z, tau)
        np.testing.assert_array_equal(r, (m > tau).sum(axis=1))
    # adding a constant to a row's logits changes nothing
    m2, _, _ = oracle.soft_gate(x, z + 7.0)
    np.testing.assert_allclose(m2, m, atol=1e-14)


def test_image_eviction_keeps_exactly_the_listed_tokens_in_order():
    # After an eviction the survivors of every (side, class) can be found again, in their arrival order, directly
    # behind one another from the key's first tile on; their rows, ranks, positions and K <-> V links are intact, the
    # rows behind the last one are zero, emptied tiles are off the lists, other sequences are untouched, and a later
    # append lands behind the survivors.
    rng = np.random.default_rng(41)
    d, S, n = 256, 3, 900
    ranks = rng.integers(1, d + 1, size=(n, 2)).astype(np.int32)
    xk = rng.integers(1, 2 ** 16, size=(n, d)).astype(np.uint16)
    xv = rng.integers(1, 2 ** 16, size=(n, d)).astype(np.uint16)
    seq = rng.integers(0, S, n).astype(np.int32)
    pos = rng.permutation(5000)[:n].astype(np.int32)
    img = CacheImage(1, d, S, 1024, 4096)
    assert img.append(0, xk[:700], xv[:700], seq[:700], pos[:700], ranks[:700])
    ref = CacheImage(1, d, S, 1024, 4096)
    assert ref.append(0, xk[:700], xv[:700], seq[:700], pos[:700], ranks[:700])
    keep = rng.permutation(pos[:700][seq[:700] == 1])[:60]
    img.evict(0, 1, np.concatenate([keep, [4999999]]))
    alive = np.zeros(n, bool); alive[:700] = (seq[:700] != 1) | np.isin(pos[:700], keep)
    assert img.append(0, xk[700:], xv[700:], seq[700:], pos[700:], ranks[700:])
    alive[700:] = True
    cls = -(-ranks // PANEL)
    assert img.seq_tokens[0, 1] == int((alive & (seq == 1)).sum())
    listed = [set(t for c in range(img.NC) for t in img.kclass_tiles[0][c]), set(t for s in range(S) for t in img.seq_vtiles[0][s])]
    for side, x in ((0, xk), (1, xv)):
        seen = {}
        for i in np.nonzero(alive)[0]:
            k = img.key(side, int(seq[i]), int(cls[i, side]))
            g = seen.get(k, 0); seen[k] = g + 1
            tid = img.key_tiles[0][k][g // TILE]; slot = g % TILE
            s_, c_, nv, base = img.tile_desc[0, side, tid]
            assert s_ == seq[i] and c_ == cls[i, side] and slot < nv and tid in listed[side]
            row = np.concatenate([img.blocks[base + j, slot * PANEL:(slot + 1) * PANEL] for j in range(c_)])
            r = ranks[i, side]
            np.testing.assert_array_equal(row[:r], x[i, :r])
            assert not row[r:].any() and img.tile_rank[0, side, tid, slot] == r
            link = img.tile_aux[0, side, tid, slot]
            assert (link if side == 0 else img.tile_aux[0, 0, link // TILE, link % TILE]) == pos[i]
        for k, g in seen.items():
            assert img.fill[0, k] == g and len(img.key_tiles[0][k]) == -(-g // TILE)
            tid = img.key_tiles[0][k][-1]
            base, c_ = img.tile_desc[0, side, tid, 3], img.tile_desc[0, side, tid, 1]
            if g % TILE:
                assert not any(img.blocks[base + j, (g % TILE) * PANEL:].any() for j in range(c_))
        # every listed tile belongs to a key's current tile run; nothing of a dropped token is reachable
        assert listed[side] == set(t for k in range(side * S * img.NC, (side + 1) * S * img.NC) for t in img.key_tiles[0][k])
    # the other sequences' tiles did not change by the eviction itself
    for side in range(2):
        for tid in range(int(ref.n_tiles[0, side])):
            if ref.tile_desc[0, side, tid, 0] != 1 and ref.tile_desc[0, side, tid, 2] == TILE:
                base, c_ = ref.tile_desc[0, side, tid, 3], ref.tile_desc[0, side, tid, 1]
                np.testing.assert_array_equal(img.blocks[base:base + c_], ref.blocks[base:base + c_])
