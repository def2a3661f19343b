"""The N > 1 path of the benchmark is "independent replicas + timing protocol".  Its host logic
runs here on CPU with the gloo backend, world size 2 (no GPU needed)."""
import json
import os
import subprocess
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    from paper_2609_24519_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.world() == (rank, world)
    replicas.barrier()
    # rank r reports (10 + 5 r) ms and (r + 1) * 100 units
    ms, units = replicas.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    tput = replicas.throughput(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    out.put((rank, ms, units, tput))
    replicas.barrier()
    dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sum_of_units_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, units, tput in res:
        assert ms == 15.0 and units == 300.0 and tput == pytest.approx(300.0 / 0.015)


def test_single_process_is_the_identity():
    from paper_2609_24519_b200 import replicas
    assert replicas.world() == (0, 1)
    assert replicas.aggregate(3.0, 7.0) == (3.0, 7.0)


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    """`bench.py --impl reference` launched the way the driver launches N > 1: rank 0 times the
    CPU oracle and prints the JSON line, the other rank exits 0 without work."""
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus",
           "2", "--steps", "1", "--warmup", "0", "--size", "256"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
