"""The N>1 path of the benchmark is 'replicas only': ranks run the same step on their own GPU and rank 0
reports units of all ranks over the slowest rank's time.  The reduction is exercised here with two gloo
ranks on the CPU, once in-process and once through the launcher that `bench.py --gpus N` itself uses."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [10.0 + rank, 3.0 - rank]                  # rank 1 is slower on the first figure, faster on the second
    red = bench.max_over_ranks(ms, dist, "cpu")
    dist.barrier()
    if rank == 0:
        out.put((red, bench.aggregate_throughput(1000.0, world, red[0])))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_max_time_and_summed_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    red, thr = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert red == [11.0, 3.0]
    assert abs(thr - 2 * 1000.0 / 11e-3) < 1e-6


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None) == [1.5, 2.5]
    assert bench.aggregate_throughput(10.0, 1, 1000.0) == 10.0


def test_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` outside a torchrun launch re-executes itself as two ranks; here with the host-side
    self-test (gloo on CPU) in place of the GPU step: rank 0 prints one line with n_gpus = 2, the slowest rank's time
    and the units of both ranks."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-selftest"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-1000:] + r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                  # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 11.0
    assert abs(lines[0]["value"] - 2 * 1000.0 / 11e-3) < 1e-6


def test_launcher_command_shape():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "2"], port=29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "4", "--steps", "2"]
