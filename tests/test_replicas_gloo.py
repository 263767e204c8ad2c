"""Multi-GPU runs are N independent replicas (no data-path collective): the only cross-rank step is
the max over ranks of the timed regions. Covered here with two gloo ranks on the CPU."""
import argparse
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r measured 10 + r ms for the resident run and 20 - r ms end to end
        got = bench.max_over_ranks([10.0 + rank, 20.0 - rank], "cpu", world)
        out[rank] = got
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_timed_regions_take_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == [11.0, 20.0] and out[1] == [11.0, 20.0]


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks([3.5, 4], "cpu", 1) == [3.5, 4.0]


def test_whole_job_throughput_counts_every_replica():
    # 2 replicas x 5 chunks within 11 ms
    assert abs(bench.replica_throughput(2, 5, 11.0) - 10 / 0.011) < 1e-9
    assert abs(bench.replica_throughput(1, 20, 1000.0) - 20.0) < 1e-12


def test_reference_arm_runs_on_rank_zero_only(capsys):
    args = argparse.Namespace(gpus=2, steps=1, warmup=0)
    assert bench.run_reference(args, 1, 2) is None
    assert capsys.readouterr().out == ""
