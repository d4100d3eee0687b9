"""The N > 1 path of bench.py on CPU: two gloo ranks check the pieces that do not need a GPU.  The (b,h)
units are independent, so ranks share no data: each draws its own inputs, times its own calls, and the
job's number is all ranks' units over the slowest rank's time (one max-reduce, no data-path collective).
The reference arm must run on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2407_12077_b200 import synth
    # each rank's slowest-time contribution: rank r pretends its region took 10 + 5 r ms
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    # ranks draw different inputs for the same call index
    a = synth.make_dense(1, 8, 2, 64, "bf16", seed=bench.rank_seed(rank, 3))
    digest = float(a.r.float().sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, digest)
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"ms": ms, "digests": gathered, "value": bench.whole_job_value(1000, world, ms)}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_whole_job_value(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["ms"] == 15.0                                   # the max over ranks, on every rank
        assert abs(r["value"] - 1000 * world / 15e-3) < 1e-6     # all ranks' units over the slowest time
        assert r["digests"][0] != r["digests"][1]                # independent inputs per rank
    assert res[0]["digests"] == res[1]["digests"]


def test_reference_arm_prints_one_line_from_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", OMP_NUM_THREADS="2")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--seq-len", "256"]
    out1 = subprocess.run(cmd, env=dict(env, RANK="1"), capture_output=True, text=True, timeout=300)
    assert out1.returncode == 0 and out1.stdout.strip() == ""
    out0 = subprocess.run(cmd, env=dict(env, RANK="0"), capture_output=True, text=True, timeout=300)
    assert out0.returncode == 0, out0.stderr
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
