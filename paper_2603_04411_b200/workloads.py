"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws inputs (states, bases, queries, gate logits, forced
ranks).  It contains none of the compression or attention arithmetic and is
imported both by the tests that feed the CPU oracle and by the GPU benchmark,
so both sides see the same buffers.

The paper evaluates on Llama-3-8B / Qwen3-8B with trained gates and text
datasets; neither is available offline, so these draws stand in for them:
shapes follow Llama-3-8B (8 KV heads x 128, GQA 4), rank statistics follow the
paper's operating points (overall Retain Rate 8.5 % .. 47 %) and its allocation
analysis (attention-sink tokens keep most components, most tokens keep few).

All tensors are torch tensors on `device`; 16-bit states are returned in the
model dtype (torch.float16 / torch.bfloat16).
"""
from dataclasses import dataclass, field

import torch

RANK_LEVELS = (1024, 512, 256, 128)     # "16/8/4/2-bit" levels: bits = 16 r / d_kv at d_kv = 1024


@dataclass
class LayerInputs:
    """Inputs of one layer: what the library's caller owns."""
    dtype: torch.dtype
    d_kv: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    Uinv_k: torch.Tensor            # [d_kv, d_kv] 16-bit, row j = spectral index j
    Uinv_v: torch.Tensor
    xt_k: torch.Tensor              # [n_tok, d_kv] 16-bit spectral states x~ (pre-RoPE)
    xt_v: torch.Tensor
    seq_ids: torch.Tensor           # [n_tok] int32
    positions: torch.Tensor         # [n_tok] int32
    q: torch.Tensor                 # [n_seq, n_q_heads, head_dim] 16-bit, already rotated
    ranks: torch.Tensor = None      # [n_tok, 2] uint16 stored as int32 tensor (forced mode) or None
    logits: torch.Tensor = None     # [n_tok, 2, d_kv] fp32 (logits mode) or None
    raw_k: torch.Tensor = None      # [n_tok, d_kv] fp64 raw states x (only kept on request)
    raw_v: torch.Tensor = None
    U_k: torch.Tensor = None        # fp64 bases (only kept on request)
    U_v: torch.Tensor = None
    extra: dict = field(default_factory=dict)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def outlier_channels(seed: int, d_kv: int, n: int) -> torch.Tensor:
    g = _gen(seed + 7919, "cpu")
    return torch.randperm(d_kv, generator=g)[:n]


def raw_states(seed: int, n_tok: int, d_kv: int, device="cpu", k_outliers=None,
               k_outlier_scale=10.0, heavy_tail=False, chunk=65536):
    """x_K, x_V ~ N(0,1) per channel (fp32); chosen K channels are scaled (x10), or, with
    heavy_tail, multiplied by |Student-t(3)| draws x 10 per token."""
    g = _gen(seed, device)
    xk = torch.empty(n_tok, d_kv, dtype=torch.float32, device=device)
    xv = torch.empty(n_tok, d_kv, dtype=torch.float32, device=device)
    for lo in range(0, n_tok, chunk):
        hi = min(n_tok, lo + chunk)
        xk[lo:hi] = torch.randn(hi - lo, d_kv, generator=g, device=device)
        xv[lo:hi] = torch.randn(hi - lo, d_kv, generator=g, device=device)
        if k_outliers is not None and len(k_outliers) > 0:
            ch = k_outliers.to(device)
            if heavy_tail:
                z = torch.randn(hi - lo, len(ch), generator=g, device=device)
                chi = torch.randn(hi - lo, len(ch), 3, generator=g, device=device).pow(2).sum(-1)
                t3 = z / torch.sqrt(chi / 3.0)
                xk[lo:hi, ch] = k_outlier_scale * t3
            else:
                xk[lo:hi, ch] *= k_outlier_scale
    return xk, xv


def pca_basis(x_calib: torch.Tensor) -> torch.Tensor:
    """Eigenvectors of the covariance of calibration states, columns sorted by
    descending eigenvalue (the paper's initialisation of U), in fp64 on the CPU."""
    x = x_calib.to(torch.float64).cpu()
    x = x - x.mean(0, keepdim=True)
    cov = (x.T @ x) / max(1, x.shape[0] - 1)
    w, v = torch.linalg.eigh(cov)
    order = torch.argsort(w, descending=True)
    return v[:, order].contiguous()


def synthetic_spectral_states(x: torch.Tensor, U: torch.Tensor, dtype, chunk=65536) -> torch.Tensor:
    """Draws the spectral states the library's boundary takes: the raw draw expressed in the calibration basis and
    rounded to the storage type.  This only gives the synthetic input its spectrum (energy concentrated in the leading
    components, like states seen through a PCA basis); it is not the library's or the oracle's Eq. 1, which are
    twkv_project and oracle.project + narrow16 and are tested against each other on raw states."""
    out = torch.empty(x.shape[0], U.shape[1], dtype=dtype, device=x.device)
    Ud = U.to(device=x.device, dtype=torch.float32)
    for lo in range(0, x.shape[0], chunk):
        hi = min(x.shape[0], lo + chunk)
        out[lo:hi] = (x[lo:hi].to(torch.float32) @ Ud).to(dtype)
    return out


def forced_ranks(seed: int, n_tok: int, levels=RANK_LEVELS, probs=None, device="cpu") -> torch.Tensor:
    """Ranks drawn from `levels` with probabilities `probs` (uniform if None); r_K = r_V."""
    g = _gen(seed + 104729, "cpu")
    if probs is None:
        idx = torch.randint(0, len(levels), (n_tok,), generator=g)
    else:
        idx = torch.multinomial(torch.tensor(probs, dtype=torch.float64), n_tok, replacement=True, generator=g)
    r = torch.tensor(levels, dtype=torch.int32)[idx]
    return torch.stack([r, r], dim=1).to(device)


def importance(seed: int, n_tok_per_seq: int, n_seq: int, device="cpu") -> torch.Tensor:
    """Heavy-tailed synthetic per-token importance u_t = exp(N(0,1)), [n_seq, T]."""
    g = _gen(seed + 15485863, device)
    return torch.exp(torch.randn(n_seq, n_tok_per_seq, generator=g, device=device))


def gate_logits(seed: int, kappa_k: torch.Tensor, kappa_v: torch.Tensor, d_kv: int,
                width=8.0, noise=0.5, chunk=32768) -> torch.Tensor:
    """Logits whose softmax peaks near truncation index d + 1 - kappa (1-based):
    z[t, j] = -|j - (d + 1 - kappa_t)| / width + noise * N(0, 1).  Returns [n, 2, d] fp32."""
    device = kappa_k.device
    n = kappa_k.shape[0]
    g = _gen(seed + 32452843, device)
    out = torch.empty(n, 2, d_kv, dtype=torch.float32, device=device)
    j = torch.arange(1, d_kv + 1, device=device, dtype=torch.float32)[None, :]
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        for side, kap in ((0, kappa_k), (1, kappa_v)):
            centre = (d_kv + 1 - kap[lo:hi].to(torch.float32))[:, None]
            z = -(j - centre).abs() / width
            z = z + noise * torch.randn(hi - lo, d_kv, generator=g, device=device)
            out[lo:hi, side] = z
    return out


def safe_logit_row(d_kv: int, kappa: int) -> torch.Tensor:
    """A logit row whose cumulative softmax jumps from ~0 to ~1 at one index
    (every cumulative sum is far from any threshold in (1e-6, 1 - 1e-6))."""
    z = torch.full((d_kv,), -40.0, dtype=torch.float32)
    z[d_kv - int(kappa)] = 0.0
    return z


def build_layer(seed: int, *, n_seq: int, ctx: int, n_q_heads: int, n_kv_heads: int = 8,
                head_dim: int = 128, dtype=torch.float16, device="cpu",
                outlier: str = "x10:4", mode: str = "forced", level_probs=None,
                mean_rank: int = 256, n_calib: int = 8192, keep_raw: bool = False,
                shuffle_positions: bool = False, rank_recipe: str = "levels") -> LayerInputs:
    """One layer of synthetic inputs: n_seq sequences of ctx tokens, tokens stored
    sequence-major (all tokens of sequence 0, then sequence 1, ...)."""
    d_kv = n_kv_heads * head_dim
    n_tok = n_seq * ctx
    kind, _, cnt = outlier.partition(":")
    if kind == "x10":
        n_out = int(cnt)
        heavy = False
    elif kind == "pct":
        n_out = max(1, int(round(d_kv * float(cnt) / 100.0)))
        heavy = False
    elif kind == "t3pct":
        n_out = max(1, int(round(d_kv * float(cnt) / 100.0)))
        heavy = True
    else:
        n_out, heavy = 0, False
    ch = outlier_channels(seed, d_kv, n_out)
    # bases from a calibration draw of the same distribution
    ck, cv = raw_states(seed + 1, n_calib, d_kv, device=device, k_outliers=ch, heavy_tail=heavy)
    U_k = pca_basis(ck)
    U_v = pca_basis(cv)
    del ck, cv
    xk, xv = raw_states(seed + 2, n_tok, d_kv, device=device, k_outliers=ch, heavy_tail=heavy)
    xt_k = synthetic_spectral_states(xk, U_k, dtype)
    xt_v = synthetic_spectral_states(xv, U_v, dtype)
    Uinv_k = U_k.T.contiguous().to(dtype).to(device)      # orthogonal basis: U^-1 = U^T
    Uinv_v = U_v.T.contiguous().to(dtype).to(device)
    g = _gen(seed + 3, "cpu")
    q = torch.randn(n_seq, n_q_heads, head_dim, generator=g).to(dtype).to(device)
    seq_ids = torch.arange(n_seq, dtype=torch.int32).repeat_interleave(ctx).to(device)
    if shuffle_positions:
        pos = torch.stack([torch.randperm(ctx, generator=g) for _ in range(n_seq)]).reshape(-1).to(torch.int32)
    else:
        pos = torch.arange(ctx, dtype=torch.int32).repeat(n_seq)
    positions = pos.to(device)
    out = LayerInputs(dtype=dtype, d_kv=d_kv, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                      head_dim=head_dim, Uinv_k=Uinv_k, Uinv_v=Uinv_v, xt_k=xt_k, xt_v=xt_v,
                      seq_ids=seq_ids, positions=positions, q=q)
    if keep_raw:
        out.raw_k, out.raw_v, out.U_k, out.U_v = xk.to(torch.float64), xv.to(torch.float64), U_k, U_v
    if mode == "forced":
        if rank_recipe == "levels":
            out.ranks = forced_ranks(seed, n_tok, probs=level_probs, device=device)
        elif rank_recipe == "sink_recent":
            # 5 % full rank: first 64 tokens and the most recent ones; the rest 256 / 128 by importance
            u = importance(seed, ctx, n_seq, device="cpu")
            n_full = int(round(0.05 * ctx))
            r = torch.where(u > u.median(dim=1, keepdim=True).values, 256, 128).to(torch.int32)
            r[:, :min(64, ctx)] = d_kv
            r[:, ctx - max(0, n_full - 64):] = d_kv
            r = r.reshape(-1)
            out.ranks = torch.stack([r, r], dim=1).to(device)
        elif rank_recipe == "any":
            # every rank 1..d_kv possible, K and V independent (stress case)
            rr = torch.randint(1, d_kv + 1, (n_tok, 2), generator=g, dtype=torch.int32)
            out.ranks = rr.to(device)
        else:
            raise ValueError(rank_recipe)
    elif mode == "logits":
        u = importance(seed, ctx, n_seq, device=device)
        kap = (mean_rank * u / 1.6487212707).clamp(1, d_kv)        # E[exp(N(0,1))] = e^0.5
        kap[:, :min(4, ctx)] = 0.75 * d_kv                          # attention sinks keep ~75 %
        gj = _gen(seed + 4, device)
        jitter = torch.exp(0.1 * torch.randn(n_seq, ctx, generator=gj, device=device))
        kap_k = kap.reshape(-1)
        kap_v = (kap * jitter).clamp(1, d_kv).reshape(-1)
        out.logits = gate_logits(seed, kap_k.round(), kap_v.round(), d_kv)
    else:
        raise ValueError(mode)
    return out


# The five benchmark configurations (shapes only; `scale` shrinks contexts for tests).
def config(i: int, device="cpu", ctx=None, n_seq=None, keep_raw=False) -> LayerInputs:
    if i == 1:
        return build_layer(0, n_seq=n_seq or 1, ctx=ctx or 1024, n_q_heads=8, dtype=torch.float16,
                           device=device, outlier="x10:4", mode="forced", keep_raw=keep_raw)
    if i == 2:
        return build_layer(1, n_seq=n_seq or 16, ctx=ctx or 32768, n_q_heads=32, dtype=torch.float16,
                           device=device, outlier="pct:1", mode="logits", mean_rank=256, keep_raw=keep_raw)
    if i == 3:
        return build_layer(2, n_seq=n_seq or 64, ctx=ctx or 8192, n_q_heads=32, dtype=torch.float16,
                           device=device, outlier="pct:1", mode="forced",
                           level_probs=(0.10, 0.20, 0.40, 0.30), shuffle_positions=True, keep_raw=keep_raw)
    if i == 4:
        return build_layer(3, n_seq=n_seq or 1, ctx=ctx or 131072, n_q_heads=64, dtype=torch.bfloat16,
                           device=device, outlier="t3pct:1", mode="forced", rank_recipe="sink_recent",
                           keep_raw=keep_raw)
    if i == 5:
        g = _gen(4, "cpu")
        e = -torch.log(torch.rand(4, generator=g))                 # Dirichlet(1,1,1,1) via exponentials
        mix = (e / e.sum()).tolist()
        return build_layer(4, n_seq=n_seq or 32, ctx=ctx or 16384, n_q_heads=32, dtype=torch.float16,
                           device=device, outlier="pct:1", mode="forced", level_probs=tuple(mix),
                           keep_raw=keep_raw)
    raise ValueError(i)


def gate_params(seed: int, d_kv: int, dtype, device="cpu", n_bumps: int = 64, first_dim: int = 64,
                gain: float = 8.0, r_min: int = 7):
    """Synthetic gate parameters (W, b) of the linear layer in front of the softmax.

    Row first_dim + k of W carries a narrow bump centred on truncation index d + 1 - r_k, with
    r_k geometric between r_min and d, so the largest of n_bumps spectral components of a
    token decides which bump wins the softmax.  The resulting ranks are spread over
    r_min .. d with a mean near d / 4, like the paper's ~25 % Retain Rate operating point.
    Returns (W_k, W_v, b_k, b_v): W [d, d] in `dtype`, b [d] fp32."""
    g = _gen(seed + 49979687, "cpu")
    j = torch.arange(1, d_kv + 1, dtype=torch.float64)
    out = []
    for side in range(2):
        W = torch.zeros(d_kv, d_kv, dtype=torch.float64)
        rk = r_min * (d_kv / r_min) ** (torch.arange(n_bumps, dtype=torch.float64) / (n_bumps - 1))
        rk = rk.round().clamp(1, d_kv)
        perm = torch.randperm(n_bumps, generator=g)
        for k in range(n_bumps):
            centre = d_kv + 1 - rk[perm[k]]
            W[first_dim + k] = gain * torch.exp(-(j - centre).abs() / 2.0)
        out.append(W.to(dtype).to(device))
    b = [(0.1 * torch.randn(d_kv, generator=g)).to(torch.float32).to(device) for _ in range(2)]
    return out[0], out[1], b[0], b[1]
