"""Timings of libtwkv on the other benchmark shapes (bench.py at the repository root times the 32k-context one).

  python -m paper_2603_04411_b200.config_bench --config 3   high-batch serving: B 64, context 8192, skewed rank mix,
                                                            shuffled positions; prefill compress, then 32 decode steps
                                                            that each append and compress one token per sequence
  python -m paper_2603_04411_b200.config_bench --config 4   long context: B 1, 64 query heads, context 131072, bf16;
                                                            one decode step per V-side split factor
  python -m paper_2603_04411_b200.config_bench --config 5   32-layer decode step, B 32, context 16384, per-layer rank
                                                            mixes; every step appends one token per sequence and runs
                                                            attention in every layer (the layers share one set of
                                                            synthetic states and bases; each has its own cache)

Inputs are seeded and synthetic (workloads.py); ranks are given (FORCED mode), as in those configurations.
One JSON line per run, times from CUDA events on the launching stream.
"""
import argparse
import json

import torch

from . import build as lib_build


def _events(n):
    return [torch.cuda.Event(enable_timing=True) for _ in range(n)]


def config3(B, workloads, dev, steps=32):
    S, CTX, HQ = 64, 8192, 32
    tot = CTX + steps
    li = workloads.build_layer(2, n_seq=S, ctx=tot, n_q_heads=HQ, dtype=torch.float16, device=dev, outlier="pct:1",
                               mode="forced", level_probs=(0.10, 0.20, 0.40, 0.30), shuffle_positions=True)
    idx = torch.arange(S * tot, device=dev).reshape(S, tot)
    pre = idx[:, :CTX].reshape(-1)
    cfg = B.make_config(n_layers=1, n_q_heads=HQ, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float16,
                        max_seqs=S, max_tokens_per_seq=tot)
    lv = li.ranks.to(torch.int16).contiguous()
    payload = int((-(-li.ranks.long() // 64) * 128).sum().item())
    pool = torch.empty(B.twkv_cache_required_bytes(cfg, payload), dtype=torch.uint8, device=dev)
    cache = B.twkv_cache_create(cfg, pool)
    B.twkv_cache_set_layer_params(cache, 0, li.Uinv_k, li.Uinv_v)
    sel = lambda t, j: t[j].contiguous()
    pk, pv, ps, pp, pl = (sel(t, pre) for t in (li.xt_k, li.xt_v, li.seq_ids, li.positions, lv))
    app = [tuple(sel(t, idx[:, CTX + s]) for t in (li.xt_k, li.xt_v, li.seq_ids, li.positions, lv)) for s in range(steps)]
    sid = torch.arange(S, dtype=torch.int32, device=dev)
    out = torch.empty(S, HQ, 128, dtype=torch.float16, device=dev)
    e = _events(2 + 2 * steps)
    torch.cuda.synchronize()
    e[0].record()
    B.twkv_compress(cache, 0, pk, pv, ps, pp, None, pl, B.TWKV_GATE_FORCED)
    e[1].record()
    for s, (xk, xv, sq, po, l) in enumerate(app):
        B.twkv_compress(cache, 0, xk, xv, sq, po, None, l, B.TWKV_GATE_FORCED)
        e[2 + 2 * s].record()
        B.twkv_decode_attn(cache, 0, li.q, sid, out)
        e[3 + 2 * s].record()
    torch.cuda.synchronize()
    assert B.twkv_cache_status(cache) == B.TWKV_OK
    t_app = sum(e[1 + 2 * s].elapsed_time(e[2 + 2 * s]) for s in range(steps)) / steps
    t_dec = sum(e[2 + 2 * s].elapsed_time(e[3 + 2 * s]) for s in range(steps)) / steps
    st = B.twkv_cache_stats(cache, 0)
    B.twkv_cache_destroy(cache)
    return {"workload": "high-batch_B64_ctx8192_gqa4_fp16_mix10-20-40-30", "prefill_compress_ms": e[0].elapsed_time(e[1]),
            "prefill_compress_tokens_per_s": S * CTX / (e[0].elapsed_time(e[1]) * 1e-3), "append_compress_ms_per_step": t_app,
            "decode_ms_per_step": t_dec, "decode_kv_tokens_per_s": st.tokens / (t_dec * 1e-3), "steps": steps,
            "retain_rate_k": st.retain_rate_k, "bytes_stored": st.bytes_stored}


def config4(B, workloads, dev):
    li = workloads.config(4, device=dev)
    S, CTX, HQ = 1, 131072, 64
    cfg = B.make_config(n_layers=1, n_q_heads=HQ, n_kv_heads=8, dtype=torch.bfloat16, out_dtype=torch.float32,
                        max_seqs=S, max_tokens_per_seq=CTX)
    payload = int((-(-li.ranks.long() // 64) * 128).sum().item())
    pool = torch.empty(B.twkv_cache_required_bytes(cfg, payload), dtype=torch.uint8, device=dev)
    cache = B.twkv_cache_create(cfg, pool)
    B.twkv_cache_set_layer_params(cache, 0, li.Uinv_k, li.Uinv_v)
    e = _events(2)
    e[0].record()
    B.twkv_compress(cache, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, li.ranks.to(torch.int16).contiguous(), B.TWKV_GATE_FORCED)
    e[1].record()
    sid = torch.zeros(1, dtype=torch.int32, device=dev)
    out = torch.empty(S, HQ, 128, dtype=torch.float32, device=dev)
    sweep = {}
    for splits in (1, 2, 4, 8, 16, 32, 64, 128, 256, 0):
        for _ in range(3):
            B.twkv_decode_attn(cache, 0, li.q, sid, out, splits)
        a, b = _events(2)
        a.record()
        for _ in range(10):
            B.twkv_decode_attn(cache, 0, li.q, sid, out, splits)
        b.record()
        torch.cuda.synchronize()
        sweep["auto" if splits == 0 else str(splits)] = a.elapsed_time(b) / 10
    assert B.twkv_cache_status(cache) == B.TWKV_OK
    st = B.twkv_cache_stats(cache, 0)
    B.twkv_cache_destroy(cache)
    best = min(sweep.values())
    return {"workload": "long-context_B1_ctx131072_gqa8_bf16_sink-recent", "compress_ms": e[0].elapsed_time(e[1]),
            "decode_ms_by_num_splits": sweep, "decode_kv_tokens_per_s_best": CTX / (best * 1e-3),
            "retain_rate_k": st.retain_rate_k, "bytes_stored": st.bytes_stored}


def config5(B, workloads, dev, layers=32, steps=4):
    S, CTX, HQ = 32, 16384, 32
    tot = CTX + steps
    g = torch.Generator().manual_seed(4)
    li = workloads.build_layer(4, n_seq=S, ctx=tot, n_q_heads=HQ, dtype=torch.float16, device=dev, outlier="pct:1", mode="forced")
    idx = torch.arange(S * tot, device=dev).reshape(S, tot)
    pre = idx[:, :CTX].reshape(-1)
    cfg = B.make_config(n_layers=layers, n_q_heads=HQ, n_kv_heads=8, dtype=torch.float16, out_dtype=torch.float16,
                        max_seqs=S, max_tokens_per_seq=tot)
    ranks = []
    for _ in range(layers):                                          # per-layer mix ~ Dirichlet(1, 1, 1, 1) over the four ranks
        ex = -torch.log(torch.rand(4, generator=g))
        r = workloads.forced_ranks(int(torch.randint(1 << 30, (1,), generator=g)), S * tot, probs=tuple((ex / ex.sum()).tolist()), device=dev)
        ranks.append(r.to(torch.int16).contiguous())
    payload = sum(int((-(-r.long() // 64) * 128).sum().item()) for r in ranks)
    pool = torch.empty(B.twkv_cache_required_bytes(cfg, payload), dtype=torch.uint8, device=dev)
    cache = B.twkv_cache_create(cfg, pool)
    sel = lambda t, j: t[j].contiguous()
    pk, pv, ps, pp = (sel(t, pre) for t in (li.xt_k, li.xt_v, li.seq_ids, li.positions))
    for l in range(layers):
        B.twkv_cache_set_layer_params(cache, l, li.Uinv_k, li.Uinv_v)
        B.twkv_compress(cache, l, pk, pv, ps, pp, None, sel(ranks[l], pre), B.TWKV_GATE_FORCED)
    app = [[tuple(sel(t, idx[:, CTX + s]) for t in (li.xt_k, li.xt_v, li.seq_ids, li.positions, ranks[l])) for l in range(layers)] for s in range(steps)]
    sid = torch.arange(S, dtype=torch.int32, device=dev)
    out = torch.empty(S, HQ, 128, dtype=torch.float16, device=dev)
    torch.cuda.synchronize()
    assert B.twkv_cache_status(cache) == B.TWKV_OK
    e = _events(steps + 1)
    e[0].record()
    for s in range(steps):
        for l in range(layers):
            xk, xv, sq, po, lv = app[s][l]
            B.twkv_compress(cache, l, xk, xv, sq, po, None, lv, B.TWKV_GATE_FORCED)
            B.twkv_decode_attn(cache, l, li.q, sid, out)
        e[s + 1].record()
    torch.cuda.synchronize()
    assert B.twkv_cache_status(cache) == B.TWKV_OK
    ms = [e[s].elapsed_time(e[s + 1]) for s in range(steps)]
    st = B.twkv_cache_stats(cache, -1)
    B.twkv_cache_destroy(cache)
    t = sum(ms[1:]) / max(1, len(ms) - 1)
    return {"workload": f"decode-step_{layers}layers_B32_ctx16384_gqa4_fp16_dirichlet-mix", "ms_per_step_all_layers": t,
            "attention_ms_per_token": t / S, "ms_per_layer": t / layers, "kv_tokens_per_s": st.tokens / (t * 1e-3),
            "steps_timed": steps - 1, "bytes_stored": st.bytes_stored, "retain_rate_k": st.retain_rate_k}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, required=True, choices=[3, 4, 5])
    args = ap.parse_args()
    lib_build.build()
    from . import binding as B, workloads
    assert torch.cuda.is_available(), "needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    res = {3: config3, 4: config4, 5: config5}[args.config](B, workloads, dev)
    res["config"] = args.config
    print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
