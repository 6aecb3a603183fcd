"""The N>1 path of bench.py on CPU: two gloo ranks, independent replicas, max-over-ranks timing."""
import os
import socket

import pytest

import numpy as np
import torch.multiprocessing as mp

from paper_2607_23264_b200 import inputs as gen, replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    assert replicas.init_process_group(world, "gloo")
    cfg = gen.MoEConfig("t", T=64, H=64, F=64, E=4, k=2, seed=3, router="xWr")
    x = replicas.rank_batch(gen.make_x(cfg), rank)
    replicas.barrier(world)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slowest = replicas.max_over_ranks(my_ms, world)
    q.put((rank, slowest, int(x[:, 0].astype(np.int64).sum()), x[0, :4].tolist()))
    replicas.barrier(world)
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_distinct_batches():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0], "every rank sees the slowest rank's time"
    assert got[0][2] == got[1][2], "same tokens, rotated"
    assert got[0][3] != got[1][3], "ranks work on different batches"
    assert replicas.job_tokens_per_second(64, world, steps=10, slowest_ms=15.0) == 64 * 2 * 10 / 0.015


def test_single_rank_needs_no_process_group():
    assert replicas.init_process_group(1, "gloo") is False
    assert replicas.max_over_ranks(3.5, 1) == 3.5
    x = np.arange(12, dtype=np.uint16).reshape(4, 3)
    assert replicas.rank_batch(x, 0) is x
    assert np.array_equal(replicas.rank_batch(x, 1), np.roll(x, 17, axis=0))


def test_launcher_command_for_two_ranks():
    cmd, env = replicas.launcher_command(2, "bench.py", ["--gpus", "2", "--steps", "5"], port=29511, python="python3")
    assert cmd[:3] == ["python3", "-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-5:] == ["bench.py", "--gpus", "2", "--steps", "5"], "the script and its own arguments come last"
    assert env == {"NCCL_DEBUG": "INFO"}
    import pytest
    with pytest.raises(ValueError):
        replicas.launcher_command(1, "bench.py", [], port=1)


def test_forced_one_rank_group_takes_the_group_path():
    """A process started by a launcher joins the group even as the only rank (gloo here, NCCL in bench.py)."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    p = ctx.Process(target=_forced_worker, args=(_free_port(), q))
    p.start()
    assert q.get(timeout=120) == (True, 7.25)
    p.join(timeout=60)
    assert p.exitcode == 0


def _forced_worker(port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1")
    import torch.distributed as dist
    joined = replicas.init_process_group(1, "gloo", force=True)
    replicas.barrier(1)
    q.put((joined and dist.is_initialized(), replicas.max_over_ranks(7.25, 1)))
    dist.destroy_process_group()


@pytest.mark.gpu
def test_bench_under_the_launcher_with_one_rank_joins_an_nccl_group():
    """bench.py started by torch.distributed.run as the only rank: NCCL group, barrier and max-over-ranks reduction on the
    GPU, the path every rank of an N-GPU run takes (N > 1 needs more GPUs than this test has)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=1", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(root, "bench.py"), "--gpus", "1", "--config", "C1",
           "--steps", "5", "--warmup", "3", "--no-cpu-baseline", "--heat-seconds", "0.2"]
    env = dict(os.environ, NCCL_DEBUG="INFO")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=root, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 1 and line["value"] > 0 and line["gpu_launches"] > 0
    assert "NCCL INFO" in (r.stdout + r.stderr), "the NCCL group was not joined"
