"""The N > 1 path of the benchmark is "replicas only": every rank runs the same chunk stream on its
own GPU, no data-path collective; the slowest rank sets the time and the bytes add up. This checks that
host logic with two gloo ranks on CPU (no GPU needed)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 5.0 - rank, 1.0]            # per-rank timings in ms
    got = bench.max_over_ranks(mine, world)
    dist.barrier()
    value = bench.job_throughput(world, 2.0e9, got[0])
    q.put((rank, got, value))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_add_their_bytes():
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
    for rank, got, value in res:
        assert got == [11.0, 5.0, 1.0]                # element-wise max over the ranks
        assert value == pytest.approx(2 * 2.0e9 / 11.0e-3 / 1e9)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1) == [3.0, 4.0]
    assert bench.job_throughput(1, 1.0e9, 1.0) == pytest.approx(1000.0)


def test_reference_arm_prints_one_json_line(tmp_path):
    """bench.py --impl reference times the CPU oracle and prints the contract's JSON line."""
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0", "--config", "1"],
                         capture_output=True, text=True, timeout=600, cwd=str(tmp_path))
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
