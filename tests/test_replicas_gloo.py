"""The multi-GPU protocol of the benchmark (independent replicas, barrier, slowest rank's
time, summed work) exercised with two gloo ranks on CPU."""

import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402

from paper_2403_20041_b200 import replicas  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier(dist)
        my_ms = 2.0 + 3.0 * rank  # rank 1 is the slow one
        slowest = replicas.max_over_ranks(my_ms, dist)
        value = replicas.whole_job_throughput(10.0, slowest * 1e-3, world)
        seeds = [None] * world
        dist.all_gather_object(seeds, replicas.rank_seed(7, rank))
        replicas.barrier(dist)
        out.put((rank, slowest, value, seeds))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_summed_work():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value, seeds in results:
        assert slowest == 5.0                      # max over ranks, on every rank
        assert value == pytest.approx(2 * 10.0 / 5e-3)
        assert len(set(seeds)) == world            # replicas draw different inputs


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_throughput(4.0, 2.0, 1) == 2.0
    replicas.barrier(None)


def test_bench_refuses_more_gpus_than_the_machine_has():
    """`python bench.py --gpus N` outside a torchrun environment starts its own ranks; on a machine with
    fewer GPUs it must fail loudly instead of running one replica and reporting n_gpus = 1."""
    import subprocess
    import sys

    import torch

    have = torch.cuda.device_count()
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", str(have + 2), "--steps", "1"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode != 0
    assert f"--gpus {have + 2}" in res.stderr and "CUDA device" in res.stderr
    assert "n_gpus" not in res.stdout


def test_bench_refuses_a_world_size_that_disagrees_with_gpus():
    import subprocess
    import sys

    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "4", "--steps", "1"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode != 0 and "WORLD_SIZE" in res.stderr
