#!/usr/bin/env python
"""Benchmark of the libtwkv hot path on the Llama-3-8B-shaped 32k-context workload.

One step = one pass of the whole hot path over one batch: reset the cache, compress all B*T
tokens (gate logits GEMM -> rank -> truncate + pack) and run one decode-attention step over the
mixed-rank cache.  The headline value is decode-attention KV tokens/s (B*T / decode time);
compress tokens/s, HBM GB/s on the compressed bytes and the per-kernel times are reported
beside it.  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
  python bench.py --config 1|3|4|5     the other synthetic workloads (tiny, high-batch serving with appends, long context
                                       with a split-K sweep, 32-layer decode step): 20 warm + at least 100 timed iterations each
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "llama3-8b-layer_B16_ctx32768_gqa4_fp16_gate-assigned-ranks"
B_SEQ, CTX, HQ, HKV, DH = 16, 32768, 32, 8, 128
D_KV = HKV * DH
METRIC = "decode_attn_kv_tokens_per_s"
UNIT = "KV tokens/s"
NOMINAL_HBM_GBS = 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "tflops": float(p["bf16_tflops"]), "tflops_sustained": float(p["bf16_tflops_sustained"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(device_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            sm.sort()
            out = {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                   "samples": len(sm), "power_w_max": max(power)}
        return out


def oracle_sample_inputs(li, gate, n_tokens):
    """Host copies of the first n_tokens of sequence 0 for the CPU oracle (fp64)."""
    import numpy as np
    import oracle
    from tests.helpers import bits16
    xk = oracle.widen16(bits16(li.xt_k[:n_tokens]), "f16")
    xv = oracle.widen16(bits16(li.xt_v[:n_tokens]), "f16")
    Wk, Wv, bk, bv = gate
    return dict(xk=xk, xv=xv, pos=li.positions[:n_tokens].cpu().numpy(),
                Uk=oracle.widen16(bits16(li.Uinv_k), "f16"), Uv=oracle.widen16(bits16(li.Uinv_v), "f16"),
                Wk=oracle.widen16(bits16(Wk), "f16"), Wv=oracle.widen16(bits16(Wv), "f16"),
                bk=bk.double().cpu().numpy(), bv=bv.double().cpu().numpy(),
                q=oracle.widen16(bits16(li.q[0]), "f16"))


def oracle_step(s, n):
    """The oracle's pass over n tokens: gate (Eq. 5, 6, 8) then decode attention.  Returns (t_gate, t_decode)."""
    import oracle
    t0 = time.perf_counter()
    rk, _ = oracle.gate_rank(oracle.gate_logits(s["xk"][:n], s["Wk"], s["bk"]), 0.1)
    rv, _ = oracle.gate_rank(oracle.gate_logits(s["xv"][:n], s["Wv"], s["bv"]), 0.1)
    t1 = time.perf_counter()
    oracle.decode_attn(s["xk"][:n], s["xv"][:n], rk, rv, s["pos"][:n], s["Uk"], s["Uv"], s["q"], HKV, 500000.0, DH ** -0.5)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def sized_oracle_sample(s, target_s, n_max):
    """Pick a token count whose oracle pass takes about target_s seconds (calibrated on 512 tokens)."""
    tg, td = oracle_step(s, 512)
    per_tok = (tg + td) / 512
    n = int(max(512, min(n_max, target_s / max(per_tok, 1e-9))))
    return n // 128 * 128


def build_workload(device):
    import torch
    from paper_2603_04411_b200 import workloads
    li = workloads.build_layer(1, n_seq=B_SEQ, ctx=CTX, n_q_heads=HQ, n_kv_heads=HKV, dtype=torch.float16,
                               device=device, outlier="pct:1", mode="forced", level_probs=None)
    li.ranks = None
    gate = workloads.gate_params(1, D_KV, torch.float16, device=device)
    return li, gate


def run_reference(args):
    import torch
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2603_04411_b200 import workloads
    n_max = 32768
    li = workloads.build_layer(1, n_seq=1, ctx=n_max, n_q_heads=HQ, n_kv_heads=HKV, dtype=torch.float16,
                               device="cpu", outlier="pct:1", mode="forced")
    gate = workloads.gate_params(1, D_KV, torch.float16)
    s = oracle_sample_inputs(li, gate, n_max)
    # the sample per step shrinks with the number of steps, so that the whole run stays within about two minutes
    n = sized_oracle_sample(s, min(4.0, 120.0 / max(args.steps, 1)), n_max)
    for _ in range(args.warmup):
        oracle_step(s, min(n, 512))
    t_dec = []
    t_all = []
    for _ in range(args.steps):
        tg, td = oracle_step(s, n)
        t_dec.append(td); t_all.append(tg + td)
    ms = 1e3 * sum(t_all) / len(t_all)
    value = n / (sum(t_dec) / len(t_dec))
    cores = oracle.num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": f"{n} tokens of one sequence, {HQ} query heads", "l2": "n/a (CPU)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"gate + decode attention over the first {n} tokens of one sequence, all {HQ} heads"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_ours(args):
    import numpy as np
    import torch

    from paper_2603_04411_b200 import build as lib_build
    lib_build.build()
    from paper_2603_04411_b200 import binding as B

    from paper_2603_04411_b200 import replicas
    world = replicas.world_size()
    rank = replicas.rank()
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init("nccl", dev)

    li, gate = build_workload(dev)
    Wk, Wv, bk, bv = gate
    n_tok = B_SEQ * CTX
    cfg = B.make_config(n_layers=1, n_q_heads=HQ, n_kv_heads=HKV, dtype=torch.float16, out_dtype=torch.float16,
                        max_seqs=B_SEQ, max_tokens_per_seq=CTX)
    pool_bytes = B.twkv_cache_required_bytes(cfg, int(n_tok * 2 * 2 * 420))     # room for mean class width ~420
    pool = torch.empty(pool_bytes, dtype=torch.uint8, device=dev)
    cache = B.twkv_cache_create(cfg, pool)
    B.twkv_cache_set_layer_params(cache, 0, li.Uinv_k, li.Uinv_v, Wk, Wv, bk, bv)
    levels = torch.zeros(n_tok, 2, dtype=torch.int16, device=dev)
    sid = torch.arange(B_SEQ, dtype=torch.int32, device=dev)
    out = torch.empty(B_SEQ, HQ, DH, dtype=torch.float16, device=dev)
    stream = torch.cuda.current_stream()

    def step(ev=None):
        B.twkv_cache_reset(cache)
        if ev: ev[0].record(stream)
        B.twkv_compress(cache, 0, li.xt_k, li.xt_v, li.seq_ids, li.positions, None, levels, B.TWKV_GATE_COMPUTE)
        if ev: ev[1].record(stream)
        B.twkv_decode_attn(cache, 0, li.q, sid, out)
        if ev: ev[2].record(stream)

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    status = B.twkv_cache_status(cache)
    assert status == B.TWKV_OK, B.twkv_status_string(status)
    st = B.twkv_cache_stats(cache, 0)
    assert st.tokens == n_tok

    B.twkv_profile_enable(cache, True)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.twkv_launch_count()
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(evs[i])
    e1.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    launches = B.twkv_launch_count() - launches0
    prof = B.twkv_profile_read(cache)
    B.twkv_profile_enable(cache, False)
    total_ms = e0.elapsed_time(e1)
    comp_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    dec_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    total_ms, comp_ms, dec_ms = replicas.max_over_ranks([total_ms, comp_ms, dec_ms], dev)
    ms_per_step = total_ms / args.steps

    # sustained leg: the same step back to back for at least two seconds with the clock sampler running, so that the
    # burst figures above can be read beside what the board holds under its power cap
    sustained = None
    if not args.skip_sustained:
        n_sus = max(args.steps, int(2200.0 / max(ms_per_step, 1e-3)))
        sampler2 = ClockSampler(local) if rank == 0 else None
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(n_sus):
            step()
        s1.record(stream)
        barrier()
        c2 = sampler2.stop() if sampler2 else None
        sus_ms = replicas.max_over_ranks([s0.elapsed_time(s1) / n_sus], dev)[0]
        if rank == 0:
            sustained = {"steps": n_sus, "ms_per_step": sus_ms, "sm_mhz_median": c2["sm_mhz"], "reasons": c2["reasons"],
                         "samples": c2["samples"], "power_w_max": c2.get("power_w_max"),
                         "ms_x_mhz": sus_ms * c2["sm_mhz"] if c2["sm_mhz"] else None}

    # end to end: host buffers in, host result out, through the same C ABI calls
    e2e = None
    n_e2e = 0 if args.skip_e2e else min(args.steps, 3)
    if n_e2e:
        h_xk = torch.empty(li.xt_k.shape, dtype=torch.float16, pin_memory=True).copy_(li.xt_k)
        h_xv = torch.empty(li.xt_v.shape, dtype=torch.float16, pin_memory=True).copy_(li.xt_v)
        h_sid = li.seq_ids.cpu().pin_memory(); h_pos = li.positions.cpu().pin_memory(); h_q = li.q.cpu().pin_memory()
        h_out = torch.empty(out.shape, dtype=out.dtype, pin_memory=True)
        d_xk, d_xv = torch.empty_like(li.xt_k), torch.empty_like(li.xt_v)
        d_sid, d_pos, d_q = torch.empty_like(li.seq_ids), torch.empty_like(li.positions), torch.empty_like(li.q)

        # The states go up in pieces of the library's own piece size on a copy stream; the compress call of a piece starts
        # when its copy has landed, so copies and kernels overlap (the cache ends up the same as after one call).
        copy_stream = torch.cuda.Stream(device=dev)
        piece = B.PIECE_TOKENS
        n_pieces = (n_tok + piece - 1) // piece
        landed = [torch.cuda.Event() for _ in range(n_pieces)]
        step_done = torch.cuda.Event()

        def e2e_step():
            copy_stream.wait_event(step_done)                     # the previous step no longer reads the device buffers
            with torch.cuda.stream(copy_stream):
                d_sid.copy_(h_sid, non_blocking=True); d_pos.copy_(h_pos, non_blocking=True); d_q.copy_(h_q, non_blocking=True)
                for p_ in range(n_pieces):
                    lo, hi = p_ * piece, min(n_tok, (p_ + 1) * piece)
                    d_xk[lo:hi].copy_(h_xk[lo:hi], non_blocking=True); d_xv[lo:hi].copy_(h_xv[lo:hi], non_blocking=True)
                    landed[p_].record(copy_stream)
            B.twkv_cache_reset(cache)
            for p_ in range(n_pieces):
                lo, hi = p_ * piece, min(n_tok, (p_ + 1) * piece)
                stream.wait_event(landed[p_])
                B.twkv_compress(cache, 0, d_xk[lo:hi], d_xv[lo:hi], d_sid[lo:hi], d_pos[lo:hi], None, levels[lo:hi], B.TWKV_GATE_COMPUTE)
            B.twkv_decode_attn(cache, 0, d_q, sid, out)
            h_out.copy_(out, non_blocking=True)
            step_done.record(stream)

        e2e_step()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        g1.record(stream)
        barrier()
        e2e_ms = replicas.max_over_ranks([g0.elapsed_time(g1) / n_e2e], dev)[0]
        h2d = sum(x.numel() * x.element_size() for x in (h_xk, h_xv, h_sid, h_pos, h_q))
        d2h = h_out.numel() * h_out.element_size()
        e2e = {"value": replicas.whole_job_rate(n_tok, e2e_ms), "unit": UNIT,
               "note": "compress + decode through the C ABI from pinned host buffers: state copies in pieces on a copy stream, each "
                       "piece compressed when it has landed, the result copied back",
               "ms_per_step": e2e_ms, "steps": n_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    if rank == 0:
        peaks = measured_peaks()
        sum_rk = st.retain_rate_k * n_tok * D_KV
        ks_ms, ks_n = prof["kscore"]
        gg_ms, gg_n = prof["gate_gemm"]
        flops_k = 2.0 * sum_rk * D_KV + n_tok * (3.0 * D_KV + 2.0 * HQ * DH)
        flops_g = 4.0 * n_tok * D_KV * D_KV                                  # both sides: 2 * (2 d^2) per token
        ks_avg_ms = ks_ms / max(ks_n, 1)
        gg_avg_ms = gg_ms / max(gg_n, 1)

        def tensor_roofline(kernel, flops, avg_ms, traffic):
            ach = flops / (avg_ms * 1e-3) / 1e12
            return {"kernel": kernel, "bound": "tensor", "achieved": ach, "peak": peaks["tflops"], "unit": "TFLOP/s",
                    "frac": ach / peaks["tflops"],
                    "peak_source": f"{peaks['source']} bf16 burst (fp16 has the same nominal rate): the tensor kernels run for 0.5-1.4 ms "
                                   f"between memory-bound ones, not back to back; against the sustained figure "
                                   f"{peaks['tflops_sustained']:.0f} the fraction is {ach / peaks['tflops_sustained']:.3f}",
                    "traffic": traffic, "flops_per_launch": flops, "avg_launch_ms": avg_ms}

        # the step's dominant kernel (largest share of the timed region) carries the `roofline` object; the dominant
        # kernel of the decode-attention half is reported beside it
        # DRAM bytes per launch from the ncu captures summarised under profiles/ (reduced cases, scaled by tokens processed)
        scale = n_tok / (16 * 32768.0)
        rl_gate = tensor_roofline("gate_tc2_kernel (tcgen05 on CTA pairs: gate logits GEMM + softmax/prefix-sum/threshold rank)", flops_g, gg_avg_ms,
                                  (577.4e6 + 364.0e6) * 4 * scale)
        rl_ks = tensor_roofline("kscore_tc_kernel (tcgen05 on CTA pairs: K reconstruct + RoPE + q.K scores)", flops_k, ks_avg_ms, (84.4e6 + 4.4e6) * 4 * scale)
        roofline = rl_gate if gg_ms >= ks_ms else rl_ks
        roofline_decode = rl_ks
        va_ms, va_n = prof["vacc"]
        pk_ms, pk_n = prof["pack"]
        bytes_v = st.bytes_stored / 2.0
        kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps} for k, v in prof.items() if v[1]}
        dec_gbs = st.bytes_stored / (dec_ms * 1e-3) / 1e9
        extra = {
            "decode_ms": dec_ms, "compress_ms": comp_ms,
            "compress_tokens_per_s": replicas.whole_job_rate(n_tok, comp_ms),
            "decode_hbm_gbs_on_stored_bytes": dec_gbs,
            "decode_hbm_frac_of_8tbs": dec_gbs / NOMINAL_HBM_GBS,
            "decode_hbm_frac_of_measured": dec_gbs / peaks["hbm_gbs"],
            "binding_bound_ms": max(st.bytes_stored / peaks["hbm_gbs"] / 1e6,
                                    (flops_k + 2.0 * HQ * (st.retain_rate_v * n_tok * D_KV)) / peaks["tflops"] / 1e9),
            "vacc_gbs": (bytes_v + n_tok * HQ * 4.0) / (va_ms / max(va_n, 1) * 1e-3) / 1e9 if va_n else None,
            "gate_gemm_tflops": (4.0 * n_tok * D_KV * D_KV) / (gg_ms / args.steps * 1e-3) / 1e12 if gg_n else None,
            # pack reads the first r elements of every row and writes the class-padded rows
            "pack_gbs": (st.bytes_algorithmic + st.bytes_stored) / (pk_ms / args.steps * 1e-3) / 1e9 if pk_n else None,
            "retain_rate_k": st.retain_rate_k, "retain_rate_v": st.retain_rate_v,
            "bytes_stored": st.bytes_stored, "bytes_algorithmic": st.bytes_algorithmic,
            "kernels": kernels,
        }
        extra["frac_of_binding_bound"] = extra["binding_bound_ms"] / dec_ms
        # the two HBM-side kernels against the measured copy bandwidth (algorithmic bytes, CUDA-event launch times)
        if extra["vacc_gbs"]:
            extra["roofline_vacc"] = {"kernel": "vacc_tc_kernel (softmax weights + absorbed V accumulate)", "bound": "hbm", "achieved": extra["vacc_gbs"],
                                      "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": extra["vacc_gbs"] / peaks["hbm_gbs"],
                                      "bytes": "stored V rows + 4 Hq bytes of scores per token",
                                      "traffic": (97.2e6 + 3.7e6) * 4 * scale}
        if extra["pack_gbs"]:
            extra["roofline_pack"] = {"kernel": "pack_kernel (truncate + pack)", "bound": "hbm", "achieved": extra["pack_gbs"],
                                      "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": extra["pack_gbs"] / peaks["hbm_gbs"],
                                      "bytes": "2 (r_K + r_V) read + class-padded rows written per token"}
        # the step before the path (Eq. 1, x~ = x U on the device), timed on its own: not part of `value` or `ms_per_step`.
        # Operand values do not change a dense product's time, so the resident states and bases stand in for x and U.
        ws = torch.empty(B.twkv_projector_required_bytes(D_KV), dtype=torch.uint8, device=dev)
        pj = B.twkv_projector_create(li.Uinv_k, li.Uinv_v, ws)
        p_k, p_v = torch.empty_like(li.xt_k), torch.empty_like(li.xt_v)
        for _ in range(3):
            B.twkv_project(pj, li.xt_k, li.xt_v, p_k, p_v)
        pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pa.record(stream)
        for _ in range(10):
            B.twkv_project(pj, li.xt_k, li.xt_v, p_k, p_v)
        pb.record(stream)
        torch.cuda.synchronize()
        assert B.twkv_projector_status(pj) == B.TWKV_OK
        B.twkv_projector_destroy(pj)
        pj_ms = pa.elapsed_time(pb) / 10
        pj_tf = 4.0 * n_tok * D_KV * D_KV / (pj_ms * 1e-3) / 1e12
        extra["project"] = {"kernel": "project_tc2_kernel (tcgen05 on CTA pairs: x~ = x U for K and V, 16-bit out by TMA store)", "ms": pj_ms,
                            "tokens_per_s": n_tok / (pj_ms * 1e-3), "achieved": pj_tf, "peak": peaks["tflops"], "unit": "TFLOP/s",
                            "frac": pj_tf / peaks["tflops"], "bound": "tensor", "timed": "10 launches back to back after the steps"}
        del p_k, p_v, ws
        # CPU baseline: the oracle as it stands on a bounded sample of the same workload
        import oracle
        cpu = None
        s = None if args.skip_cpu_baseline else oracle_sample_inputs(li, gate, CTX)
        n_s = sized_oracle_sample(s, 6.0, CTX) if s else 0
        reps, tg, td = 0, 0.0, 0.0
        while s and reps < 16 and tg + td < 12.0:              # repeat the sample until ~12 s of CPU work
            a, b = oracle_step(s, n_s)
            tg, td, reps = tg + a, td + b, reps + 1
        if s:
          cpu = {"value": reps * n_s / td, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"{reps} x decode attention over the first {n_s} tokens of sequence 0, all {HQ} heads, "
                         f"{td:.2f} s in total (the gate passes over the same tokens took {tg:.2f} s)"}
        line = {"metric": METRIC, "value": replicas.whole_job_rate(n_tok, dec_ms), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "batch": B_SEQ, "context": CTX, "n_q_heads": HQ, "n_kv_heads": HKV,
                           "head_dim": DH, "step": "cache reset + compress(COMPUTE gate) of B*T tokens + one decode-attention step",
                           "l2": "inputs_exceed_l2 (cache %.0f MB, states 2.1 GB)" % (st.bytes_stored / 1e6),
                           "sharding": "replica per GPU (independent sequences), no collective"},
                "roofline": roofline, "roofline_decode_attn": roofline_decode, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
                "sustained": sustained}
        line.update(extra)
        print(json.dumps(line), flush=True)
    B.twkv_cache_destroy(cache)
    replicas.finish()


# ------------------------------------------------------------------------------------------------------------------
# The other four workloads (`--config 1|3|4|5`): one JSON line each, same objects as the headline line.
def _median_min(xs):
    xs = sorted(xs)
    return {"median": xs[len(xs) // 2], "min": xs[0], "n": len(xs)}


def _decode_flops(st, n_tok, hq):
    """Algorithmic flops of one decode step over the cached tokens: K reconstruct 2 r_K d, RoPE 3 d, scores 2 Hq d_h,
    absorbed PV 2 Hq r_V (per token), from the cache's rank sums."""
    sum_rk, sum_rv = st.retain_rate_k * n_tok * D_KV, st.retain_rate_v * n_tok * D_KV
    k_side = 2.0 * sum_rk * D_KV + n_tok * (3.0 * D_KV + 2.0 * hq * DH)
    return k_side, k_side + 2.0 * hq * sum_rv


def _decode_report(st, n_tok, hq, dec_ms, ks_ms, peaks):
    k_flops, all_flops = _decode_flops(st, n_tok, hq)
    gbs = st.bytes_stored / (dec_ms * 1e-3) / 1e9
    bound_ms = max(st.bytes_stored / peaks["hbm_gbs"] / 1e6, all_flops / peaks["tflops"] / 1e9)
    ach = k_flops / (ks_ms * 1e-3) / 1e12
    return {"decode_kv_tokens_per_s": n_tok / (dec_ms * 1e-3), "decode_hbm_gbs_on_stored_bytes": gbs,
            "decode_hbm_frac_of_8tbs": gbs / NOMINAL_HBM_GBS, "decode_hbm_frac_of_measured": gbs / peaks["hbm_gbs"],
            "binding_bound_ms": bound_ms, "frac_of_binding_bound": bound_ms / dec_ms,
            "roofline": {"kernel": "kscore_tc_kernel (tcgen05 on CTA pairs: K reconstruct + RoPE + q.K scores)", "bound": "tensor",
                         "achieved": ach, "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": ach / peaks["tflops"],
                         "peak_source": f"{peaks['source']} bf16 burst", "traffic": None, "flops_per_launch": k_flops, "avg_launch_ms": ks_ms}}


def _oracle_decode_baseline(li, ranks, seq, n_cap, dn, hq, label, full_tokens):
    """The oracle's decode attention over (a prefix of) one sequence, timed; linear extrapolation to the whole workload."""
    import numpy as np
    import oracle
    from tests.helpers import bits16
    idx = (li.seq_ids == seq).nonzero().flatten()[:n_cap]
    w = lambda t: oracle.widen16(bits16(t), dn)
    xk, xv = w(li.xt_k[idx]), w(li.xt_v[idx])
    r = ranks[idx].cpu().numpy().astype(np.int32)
    pos = li.positions[idx].cpu().numpy()
    Uk, Uv, q = w(li.Uinv_k), w(li.Uinv_v), w(li.q[seq])
    t0 = time.perf_counter()
    oracle.decode_attn(xk, xv, r[:, 0], r[:, 1], pos, Uk, Uv, q, HKV, 500000.0, DH ** -0.5)
    dt = time.perf_counter() - t0
    n = len(idx)
    return {"value": n / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{label}: decode attention over {n} tokens of sequence {seq}, all {hq} heads, {dt:.2f} s",
            "extrapolated_s_per_step_whole_workload": full_tokens / (n / dt),
            "extrapolation": "linear in the number of cached tokens (the oracle's cost per token does not depend on the context)"}


def run_config(args):
    import numpy as np
    import torch
    from paper_2603_04411_b200 import build as lib_build
    lib_build.build()
    from paper_2603_04411_b200 import binding as B, workloads
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    ci = args.config
    # at least 20 warm + 100 timed iterations; more where a step is short, so that the timed region spans ~0.4 s and the
    # clock sampler (one nvidia-smi reading every 20 - 30 ms) sees it at least ten times
    WARM, TIMED = 20, {1: 4000, 3: 600, 4: 1500, 5: 100}[ci]
    shapes = {1: dict(S=1, ctx=1024, hq=8, dt=torch.float16, name="tiny_B1_ctx1024_mha8_fp16_uniform-levels"),
              3: dict(S=64, ctx=8192, hq=32, dt=torch.float16, name="high-batch_B64_ctx8192_gqa4_fp16_mix10-20-40-30"),
              4: dict(S=1, ctx=131072, hq=64, dt=torch.bfloat16, name="long-context_B1_ctx131072_gqa8_bf16_sink-recent"),
              5: dict(S=32, ctx=16384, hq=32, dt=torch.float16, name="decode-step_32layers_B32_ctx16384_gqa4_fp16_dirichlet-mix")}[ci]
    S, ctx, hq, dt = shapes["S"], shapes["ctx"], shapes["hq"], shapes["dt"]
    dn = "f16" if dt == torch.float16 else "bf16"
    layers = 32 if ci == 5 else 1
    appends = ci in (3, 5)
    n_app = (WARM + TIMED + 8) if appends else 0                    # appended tokens per sequence (FORCED steps + a few COMPUTE ones)
    tot = ctx + n_app
    if ci == 1:
        li = workloads.config(1, device=dev)
    elif ci == 3:
        li = workloads.build_layer(2, n_seq=S, ctx=tot, n_q_heads=hq, dtype=dt, device=dev, outlier="pct:1", mode="forced",
                                   level_probs=(0.10, 0.20, 0.40, 0.30), shuffle_positions=True)
    elif ci == 4:
        li = workloads.config(4, device=dev)
    else:
        li = workloads.build_layer(4, n_seq=S, ctx=tot, n_q_heads=hq, dtype=dt, device=dev, outlier="pct:1", mode="forced")
    g = torch.Generator().manual_seed(4)
    if ci == 5:                                                     # per-layer mix ~ Dirichlet(1, 1, 1, 1) over the four ranks
        ranks = []
        for _ in range(layers):
            ex = -torch.log(torch.rand(4, generator=g))
            ranks.append(workloads.forced_ranks(int(torch.randint(1 << 30, (1,), generator=g)), S * tot,
                                                probs=tuple((ex / ex.sum()).tolist()), device=dev).to(torch.int16).contiguous())
    else:
        ranks = [li.ranks.to(torch.int16).contiguous()]
    gate = workloads.gate_params(1, D_KV, dt, device=dev) if appends else None
    cfg = B.make_config(n_layers=layers, n_q_heads=hq, n_kv_heads=HKV, dtype=dt, out_dtype=torch.float32 if dt == torch.bfloat16 else dt,
                        max_seqs=S, max_tokens_per_seq=tot)
    payload = sum(int((-(-r.long() // 64) * 128).sum().item()) for r in ranks) + (8 * S * layers * 4096 if appends else 0)
    pool = torch.empty(B.twkv_cache_required_bytes(cfg, payload), dtype=torch.uint8, device=dev)
    cache = B.twkv_cache_create(cfg, pool)
    idx = torch.arange(S * tot, device=dev).reshape(S, tot)
    pre = idx[:, :ctx].reshape(-1)
    sel = lambda t, j: t[j].contiguous()
    pk, pv, ps, pp = (sel(t, pre) for t in (li.xt_k, li.xt_v, li.seq_ids, li.positions))
    ev = lambda: torch.cuda.Event(enable_timing=True)
    pre_ms = []
    for l in range(layers):
        if gate:
            B.twkv_cache_set_layer_params(cache, l, li.Uinv_k, li.Uinv_v, *gate)
        else:
            B.twkv_cache_set_layer_params(cache, l, li.Uinv_k, li.Uinv_v)
        a, b = ev(), ev()
        a.record()
        B.twkv_compress(cache, l, pk, pv, ps, pp, None, sel(ranks[l], pre), B.TWKV_GATE_FORCED)
        b.record()
        torch.cuda.synchronize()
        pre_ms.append(a.elapsed_time(b))
    assert B.twkv_cache_status(cache) == B.TWKV_OK
    st0 = B.twkv_cache_stats(cache, 0)
    sid = torch.arange(S, dtype=torch.int32, device=dev)
    out = torch.empty(S, hq, DH, dtype=torch.float32 if dt == torch.bfloat16 else dt, device=dev)
    res = {"metric": METRIC, "unit": UNIT, "n_gpus": 1, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dn,
           "data": "synthetic", "warmup": WARM, "steps": TIMED,
           "config": {"workload": shapes["name"], "batch": S, "context": ctx, "n_q_heads": hq, "n_kv_heads": HKV, "head_dim": DH, "layers": layers,
                      "l2": "cache fits in L2: an L2-resident number, not an HBM one" if ci == 1 else "cache exceeds L2"},
           "prefill_compress_forced_ms_per_layer": _median_min(pre_ms),
           "prefill_compress_tokens_per_s": S * ctx / (sorted(pre_ms)[len(pre_ms) // 2] * 1e-3)}

    def timed_loop(body, n_warm, n_timed):
        for i in range(n_warm):
            body(i)
        torch.cuda.synchronize()
        B.twkv_profile_enable(cache, True)
        sampler = ClockSampler(0)
        marks = [(ev(), ev()) for _ in range(n_timed)]
        launches0 = B.twkv_launch_count()
        for i in range(n_timed):
            marks[i][0].record()
            body(n_warm + i)
            marks[i][1].record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        prof = B.twkv_profile_read(cache)
        B.twkv_profile_enable(cache, False)
        return [a.elapsed_time(b) for a, b in marks], prof, clocks, B.twkv_launch_count() - launches0

    if not appends:
        sweep = None
        if ci == 4:                                               # the split-K sweep of the long-context workload
            sweep = {}
            for splits in (1, 2, 4, 8, 16, 32, 64, 128, 256, 0):
                ms, _, _, _ = timed_loop(lambda i: B.twkv_decode_attn(cache, 0, li.q, sid, out, splits), 3, 20)
                sweep["auto" if splits == 0 else str(splits)] = _median_min(ms)
        ms, prof, clocks, launches = timed_loop(lambda i: B.twkv_decode_attn(cache, 0, li.q, sid, out), WARM, TIMED)
        st = st0
        n_tok = S * ctx
        dec = _median_min(ms)
        res.update({"value": n_tok / (dec["median"] * 1e-3), "ms_per_step": dec["median"], "decode_ms": dec, "clocks": clocks,
                    "gpu_launches": int(launches), "step": "one decode-attention call over the cache"})
        res.update(_decode_report(st, n_tok, hq, dec["median"], prof["kscore"][0] / max(1, prof["kscore"][1]), peaks))
        if sweep:
            res["decode_ms_by_num_splits"] = sweep
    else:
        # the appended tokens of every step, gathered before anything is timed
        app_x = [tuple(sel(t, idx[:, ctx + s_]) for t in (li.xt_k, li.xt_v, li.seq_ids, li.positions)) for s_ in range(n_app)]
        app_r = [[sel(ranks[l], idx[:, ctx + s_]) for s_ in range(n_app)] for l in range(layers)]
        app = lambda s_, l: app_x[s_] + (app_r[l][s_],)
        dec_ms, app_ms = [], []

        def body(i):
            a, m, b = ev(), ev(), ev()
            for l in range(layers):
                xk, xv, sq, po, lv = app(i, l)
                if l == 0: a.record()
                B.twkv_compress(cache, l, xk, xv, sq, po, None, lv, B.TWKV_GATE_FORCED)
                if l == 0: m.record()
                B.twkv_decode_attn(cache, l, li.q, sid, out)
                if l == 0: b.record()
            body.marks.append((a, m, b))
        body.marks = []
        ms, prof, clocks, launches = timed_loop(body, WARM, TIMED)
        for a, m, b in body.marks[WARM:]:
            app_ms.append(a.elapsed_time(m)); dec_ms.append(m.elapsed_time(b))
        assert B.twkv_cache_status(cache) == B.TWKV_OK
        st = B.twkv_cache_stats(cache, 0)
        n_tok = int(st.tokens)
        step, dec, appf = _median_min(ms), _median_min(dec_ms), _median_min(app_ms)
        res.update({"value": n_tok * layers / (step["median"] * 1e-3) if ci == 5 else n_tok / (dec["median"] * 1e-3),
                    "ms_per_step": step["median"], "step_ms": step, "decode_ms_layer0": dec, "append_forced_ms_layer0": appf,
                    "clocks": clocks, "gpu_launches": int(launches),
                    "step": f"every layer ({layers}): append one token per sequence (FORCED ranks) + decode attention"})
        if ci == 5:
            res["attention_ms_per_generated_token"] = step["median"] / S
            res["ms_per_layer"] = step["median"] / layers
        ks_ms = prof["kscore"][0] / max(1, prof["kscore"][1])
        res.update(_decode_report(st, n_tok, hq, dec["median"], ks_ms, peaks))
        # the append with the gate computed by the library (small-call path: warp-MMA logits GEMM + rank kernel), bound by
        # reading W_K and W_V (2 x 2 MiB) and the launch chain
        cms = []
        for j in range(8):
            xk, xv, sq, po, _ = app(WARM + TIMED + j, 0)
            lv = torch.zeros(S, 2, dtype=torch.int16, device=dev)
            a, b = ev(), ev()
            a.record()
            B.twkv_compress(cache, 0, xk, xv, sq, po, None, lv, B.TWKV_GATE_COMPUTE)
            b.record()
            torch.cuda.synchronize()
            cms.append(a.elapsed_time(b))
        assert B.twkv_cache_status(cache) == B.TWKV_OK
        cm = _median_min(cms[2:])
        wbytes = 2.0 * D_KV * D_KV * 2 + 2.0 * S * D_KV * 2
        res["append_compute_gate_ms_layer0"] = cm
        res["append_compute_gate_roofline"] = {"kernel": "gate_gemm_kernel + gate_rank_kernel + alloc + pack (one call of %d tokens)" % S,
                                               "bound": "hbm", "achieved": wbytes / (cm["median"] * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                               "frac": wbytes / (cm["median"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                               "bytes": "W_K, W_V (2 x 2 MiB) + the call's states; a launch-latency-bound chain of four kernels"}
    res["retain_rate_k"], res["retain_rate_v"] = st.retain_rate_k, st.retain_rate_v
    res["bytes_stored_layer0"], res["bytes_algorithmic_layer0"] = st.bytes_stored, st.bytes_algorithmic
    if not args.skip_cpu_baseline:
        cap = {1: 1024, 3: 8192, 4: 16384, 5: 16384}[ci]
        label = {1: "the whole workload", 3: "one sequence, one step", 4: "the first 16384 tokens of the sequence", 5: "one sequence, one layer, one step"}[ci]
        rk = torch.stack([ranks[0][:, 0], ranks[0][:, 1]], dim=1)
        res["cpu_baseline"] = _oracle_decode_baseline(li, rk, 0, cap, dn, hq, label, S * ctx * layers)
    B.twkv_cache_destroy(cache)
    print(json.dumps(res), flush=True)


def main():
    global B_SEQ, CTX, WORKLOAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=150)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=B_SEQ, help="sequences (default: the benchmark workload's 16)")
    ap.add_argument("--ctx", type=int, default=CTX, help="context length (default: the benchmark workload's 32768)")
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5],
                    help="which synthetic workload: 2 (default) is the headline 32k-context step, the others print their own line")
    ap.add_argument("--skip-e2e", action="store_true", help="profiling runs: leave the host-buffer leg out")
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="profiling runs: leave the oracle leg out")
    ap.add_argument("--skip-sustained", action="store_true", help="profiling runs: leave the two-second back-to-back leg out")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand with --gpus N: launch the N ranks (one per GPU) the way the driver does and hand over
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
               "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if (args.batch, args.ctx) != (B_SEQ, CTX):
        B_SEQ, CTX = args.batch, args.ctx
        WORKLOAD = f"reduced-for-profiling_B{B_SEQ}_ctx{CTX}_gqa4_fp16_gate-assigned-ranks"
    if args.impl == "reference":
        run_reference(args)
    elif args.config != 2:
        run_config(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
