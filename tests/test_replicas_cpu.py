"""The N > 1 host path ("replicas only"): two gloo ranks on the CPU.

Every rank runs the whole path by itself; the ranks only meet at the barriers around
the timed region and in the maximum over ranks of their timings.  These tests run the
helper that bench.py uses for that with world_size 2 and the gloo backend, and check
that the CPU arm of bench.py leaves all ranks but rank 0 silent.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2012_02030_b200 import replicas  # noqa: E402


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    env = {"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world)}
    os.environ.update(env, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    info = replicas.rank_info(env)
    assert (info.rank, info.local_rank, info.world) == (rank, rank, world)
    replicas.init(info, "gloo")
    replicas.barrier(info)
    # rank r pretends its step took (10 + 5 r) ms and its forward (1 + r) ms
    mine = [10.0 + 5.0 * rank, 1.0 + rank]
    total_ms, fwd_ms = replicas.max_over_ranks(info, mine)
    units = 1000.0  # per replica, identical on all ranks (weak scaling)
    value = replicas.job_throughput(info, units, fwd_ms * 1e-3)
    replicas.barrier(info)
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"total_ms": total_ms, "fwd_ms": fwd_ms, "value": value}, f)
    replicas.shutdown(info)


def test_two_replicas_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(world)]
    for r in res:  # every rank sees the slowest rank's timings
        assert r["total_ms"] == 15.0
        assert r["fwd_ms"] == 2.0
        # two replicas' units over the slowest replica's time
        assert r["value"] == pytest.approx(2 * 1000.0 / 2.0e-3)


def test_single_process_is_rank_0_of_1():
    info = replicas.rank_info({})
    assert (info.rank, info.local_rank, info.world) == (0, 0, 1)
    replicas.init(info, "gloo")  # no process group for one replica
    assert not torch.distributed.is_initialized()
    replicas.barrier(info)
    assert replicas.max_over_ranks(info, [3.0, 4.5]) == [3.0, 4.5]
    assert replicas.job_throughput(info, 10.0, 2.0) == 5.0
    with pytest.raises(ValueError):
        replicas.job_throughput(info, 10.0, 0.0)
    replicas.shutdown(info)


def test_reference_arm_other_ranks_stay_silent():
    """Under a multi-rank launch only rank 0 runs and prints the CPU arm."""
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    assert r.stdout.strip() == ""


def test_reference_arm_rank0_line():
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert line["gpu_launches"] == 0 and line["value"] > 0
