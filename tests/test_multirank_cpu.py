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


def test_gpus_flag_starts_the_replica_processes_itself():
    """`python bench.py --gpus 2` from a plain shell (no WORLD_SIZE): the script itself starts two ranks, they
    meet over 127.0.0.1 and rank 0 alone prints the line, with n_gpus = 2 and the whole-job figure from the
    slower rank's time.  --rendezvous-only keeps the GPU work out of it (gloo, CPU)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "5", "--tokens", "512",
                          "--rendezvous-only"], capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout                      # rank 0 only
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["scaling"] == "weak"
    # slower rank: 15 ms for 5 steps; 2 ranks x 5 steps x 512 calls
    assert abs(out["ms_per_step"] - 3.0) < 1e-9
    assert abs(out["value"] - 15e3 / 5120) < 1e-9


def test_replica_launch_command_shape():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.replica_launch_command(4, ["--gpus", "4", "--steps", "2"], 29511)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")
