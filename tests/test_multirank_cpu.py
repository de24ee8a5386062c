"""The N > 1 path of bench.py on CPU: two gloo ranks, no GPU.  The path shards by replica with no
data-path collective, so what there is to check is the timing aggregation (max over ranks, whole-job
rate) and that only rank 0 of the reference arm does any work."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slowest = bench.max_over_ranks(my_ms, torch.device("cpu"), True)
    dist.barrier()
    out[rank] = (slowest, bench.whole_job_rate(world, 1000.0, slowest))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_with_two_gloo_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, 29611, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    slowest, rate = res[0]
    assert slowest == 15.0                          # the maximum, on every rank
    assert abs(rate - 2 * 1000.0 / 15e-3) < 1e-6    # units of all ranks / slowest rank's time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_rate(1, 7.0, 2.0) == 3500.0


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` with no launcher around it (WORLD_SIZE unset) starts two ranks through
    torch.distributed.run; with --dry-run-cpu they rendezvous over gloo on 127.0.0.1, take the maximum of
    their (made-up) times and rank 0 alone prints the line, with n_gpus = 2."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run-cpu", "--steps", "3",
                        "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 15.0 and line["scaling"] == "weak"
    assert abs(line["value"] - 2 / 15e-3) < 1e-9


def test_launcher_command_uses_the_loopback_rendezvous():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(["--gpus", "4", "--steps", "7"], 4, 29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--master-addr" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"]
    # a process that already is a rank never relaunches
    class A:
        gpus, impl = 4, "forge"
    os.environ["WORLD_SIZE"] = "4"
    try:
        assert bench.maybe_relaunch(A, []) is None
    finally:
        del os.environ["WORLD_SIZE"]
