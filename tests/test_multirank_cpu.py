"""The N > 1 logic of bench.py on CPU: two gloo ranks, replicas only.

The path does not shard (no data-path collective); with N GPUs each rank runs
its own replica and the only exchange is the MAX of the timing scalars.  This
test runs that exchange with world_size 2 over gloo and checks the whole-job
figure derived from it."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]          # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(local)
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_timing_is_max_over_ranks_and_value_is_whole_job():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [15.0, 100.0]
    sys.path.insert(0, ROOT)
    import bench
    # 2 ranks, 5 steps of 512 calls each in 15 ms (slowest rank): 15 ms / 5120 calls
    assert abs(bench.whole_job_us_per_call(15.0, 2, 5, 512) - 15e3 / 5120) < 1e-12
    # single process: values pass through untouched
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_reference_arm_runs_on_rank0_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    args = bench.parse.__globals__["argparse"].Namespace(gpus=2, steps=1, warmup=1, impl="reference")
    bench.run_reference(args)                                   # rank 1: returns at once, prints nothing
    assert capsys.readouterr().out == ""
