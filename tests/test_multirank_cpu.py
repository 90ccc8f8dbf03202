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


# ------------------------------------------------------------ d_ff sharding
def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    from oracle import prox_oracle as po
    from paper_2607_27591_b200 import inputs, sharded
    D, F, k1, k2 = 512, 1536, 154, 358
    wg, wu, wd, x = inputs.make_small(D, F, 3, seed=21)
    wg, wu, wd, x = [po.bf16_to_f64(a) for a in (wg, wu, wd, x)]
    # equal scores across the shard boundary: channel 900 (rank 1) is a copy of channel 100 (rank 0), and the
    # k2-th place is made to fall on that pair for token 1 (see the parent test)
    wg[900], wu[900] = wg[100], wu[100]
    lo, hi = sharded.shard_range(F, world, rank)
    qg, sg = po.quantize_proxy(wg[lo:hi], 4, 128)
    qu, su = po.quantize_proxy(wu[lo:hi], 4, 128)
    dg, du = po.dequantize(qg, sg, 128), po.dequantize(qu, su, 128)
    res = []
    for t, k2_t in ((0, k2), (1, out["k2_tie"]), (2, 1), (2, F)):
        idx = po.input_topk(x[t], k1)

        def s1(xv):
            return torch.from_numpy(po.proxy_scores(xv.numpy(), idx, dg, du).astype(np.float32))

        def s2(xv, sel):
            return torch.from_numpy(po.stage2(xv.numpy(), sel.numpy(), wg[lo:hi], wu[lo:hi], wd[:, lo:hi])[0])

        sel, y = sharded.sharded_forward(s1, s2, torch.from_numpy(x[t]), k2_t, lo)
        res.append(((sel + lo).tolist(), y.numpy().tolist()))
    out[rank] = res
    dist.destroy_process_group()


def test_dff_sharding_gives_the_single_rank_mask_and_output():
    """Two gloo ranks, each with half of the channels: the exchanged mask EQUALS the single-rank top-k2 mask, ties
    across the shard boundary included, and the all-reduced y is the single-rank y."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import prox_oracle as po
    from paper_2607_27591_b200 import inputs
    D, F, k1, k2 = 512, 1536, 154, 358
    wg, wu, wd, x = inputs.make_small(D, F, 3, seed=21)
    wg, wu, wd, x = [po.bf16_to_f64(a) for a in (wg, wu, wd, x)]
    wg[900], wu[900] = wg[100], wu[100]
    qg, sg = po.quantize_proxy(wg, 4, 128)
    qu, su = po.quantize_proxy(wu, 4, 128)
    dg, du = po.dequantize(qg, sg, 128), po.dequantize(qu, su, 128)
    # the scores as the shards see them (fp32), and the k2 for token 1 at which the tied pair straddles the cut
    sc1 = po.proxy_scores(x[1], po.input_topk(x[1], k1), dg, du).astype(np.float32).astype(np.float64)
    assert sc1[100] == sc1[900]
    k2_tie = int(np.sum(sc1 > sc1[100])) + 1                # keeps channel 100, drops its copy 900
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        out["k2_tie"] = k2_tie
        mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    for case, (t, k2_t) in enumerate(((0, k2), (1, k2_tie), (2, 1), (2, F))):
        score = po.proxy_scores(x[t], po.input_topk(x[t], k1), dg, du).astype(np.float32).astype(np.float64)
        sel_ref, _ = po.channel_topk(score, k2_t)
        got = sorted(r0[case][0] + r1[case][0])
        assert got == sel_ref.tolist(), (case, len(got))
        assert all(c < F // 2 for c in r0[case][0]) and all(c >= F // 2 for c in r1[case][0])
        y_ref = po.stage2(x[t], sel_ref, wg, wu, wd)[0]
        rms = float(np.sqrt(np.mean(y_ref ** 2)))
        for r in (r0, r1):
            assert np.max(np.abs(np.asarray(r[case][1]) - y_ref)) <= 2e-2 * rms
        assert r0[case][1] == r1[case][1]                   # the all-reduce leaves the same y on both ranks
    assert 100 in r0[1][0] and 900 not in r1[1][0]          # the tie went to the lower global channel


def test_shard_range_and_single_process_mask():
    sys.path.insert(0, ROOT)
    from paper_2607_27591_b200 import sharded
    assert sharded.shard_range(1536, 2, 1) == (768, 1536)
    try:
        sharded.shard_range(10, 4, 0)
        assert False
    except ValueError:
        pass
    s = torch.tensor([0.5, 2.0, 0.0, 2.0, 1.0, 2.0], dtype=torch.float32)
    assert sharded.global_topk_mask(s, 2, 0).tolist() == [1, 3]          # equal scores: lower channel first
    assert sharded.global_topk_mask(s, 4, 0).tolist() == [1, 3, 4, 5]
    assert sharded.global_topk_mask(s, 6, 0).tolist() == [0, 1, 2, 3, 4, 5]
