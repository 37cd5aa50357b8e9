"""The N > 1 path of the benchmark is N independent replicas: no collective touches the data, only
the timing is reduced (max over ranks).  World size 2 over gloo on CPU covers that bookkeeping."""
import os
import socket
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    import torch
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r pretends its timed region took (10 + r) ms and its end-to-end region (20 - r) ms
        got = bench.max_over_ranks([10.0 + rank, 20.0 - rank], dist, torch.device("cpu"))
        out.put((rank, got))
    finally:
        dist.destroy_process_group()


def test_timing_is_max_over_ranks_world2():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [11.0, 20.0]


def test_job_throughput_counts_all_replicas():
    sys.path.insert(0, str(ROOT))
    import bench
    seqs, us_per_seq, per_sec = bench.job_throughput(world=4, seqs_per_replica=20, ms_per_step=2.0)
    assert seqs == 80
    assert us_per_seq == pytest.approx(25.0)
    assert per_sec == pytest.approx(40000.0)
    assert bench.max_over_ranks([1.5], None, "cpu") == [1.5]


def test_reference_arm_runs_on_rank0_only(monkeypatch, capsys):
    sys.path.insert(0, str(ROOT))
    import bench

    class A:
        workload, steps, warmup, gpus = "cfg1", 1, 0, 2
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(A)
    assert capsys.readouterr().out == ""


def test_gpus_flag_alone_starts_the_ranks():
    """`bench.py --gpus 2` with no launcher around it starts two ranks itself; the bookkeeping-only mode
    (gloo, no GPU work) shows that both joined: n_gpus = 2 and the step time is the slower rank's."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--replica-check"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["ms_per_step"] == 11.0 and d["sequences_per_step"] == 2
