"""The multi-rank bookkeeping of bench.py (barrier, max over ranks, whole-job rate) on two gloo ranks on the CPU."""
import os
import socket

import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2603_04411_b200 import replicas
    replicas.init("gloo")
    replicas.barrier()
    # rank r measured (10 + r, 3 - r) ms for two regions: every rank must see the slower rank's time for each
    got = replicas.max_over_ranks([10.0 + rank, 3.0 - rank])
    rate = replicas.whole_job_rate(1000.0, got[0])
    replicas.barrier()
    replicas.finish()
    q.put((rank, got, rate))


def test_two_gloo_ranks_agree_on_max_times_and_whole_job_rate():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, rate in res:
        assert got == [11.0, 3.0]                         # max over ranks, element-wise
        assert abs(rate - 2 * 1000.0 / 11.0e-3) < 1e-6    # all ranks' units over the slowest rank's time
    assert [r for r, _, _ in res] == [0, 1]


def test_single_rank_is_a_no_op(monkeypatch):
    monkeypatch.setenv("WORLD_SIZE", "1")
    monkeypatch.setenv("RANK", "0")
    from paper_2603_04411_b200 import replicas
    replicas.init("gloo")
    replicas.barrier()
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.whole_job_rate(10.0, 5.0) == 10.0 / 5.0e-3
    replicas.finish()


def test_bench_spawns_its_ranks_when_started_by_hand():
    # `python bench.py --gpus 2` without a launcher's environment starts the two ranks itself; here through the
    # reference arm (the CPU oracle), whose rank 0 prints the line and whose other ranks leave without work
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600, env=env, cwd=root)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["metric"] == "decode_attn_kv_tokens_per_s"
    assert line["unit"] == line["e2e"]["unit"] == "KV tokens/s" and line["value"] > 0
