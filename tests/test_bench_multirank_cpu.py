"""The N > 1 logic of bench.py on CPU: two gloo ranks, the slowest rank sets the step time and the
whole-job value counts every rank's tokens (weak scaling, no data-path collective)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first timer, faster on the second
    got = bench.max_over_ranks(local)
    dist.barrier()
    if rank == 0:
        out.put(got)
    dist.destroy_process_group()


def test_max_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got == [15.0, 3.0]


def test_whole_job_value_and_single_rank_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    # 2 ranks x 1000 tokens each in 0.5 ms
    assert bench.whole_job_value(1000, 2, 0.5) == 4_000_000.0


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    args = argparse.Namespace(workload="tiny", steps=1, warmup=0, gpus=2)
    bench.run_reference(args, rank=1, world=2)
    assert capsys.readouterr().out == ""
    bench.run_reference(args, rank=0, world=2)
    import json
    line = json.loads(capsys.readouterr().out)
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "KV tokens/s"


def _run_bench(*args):
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                          timeout=600, cwd=ROOT, env=env)


def test_gpus_n_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher starts two ranks itself; they meet over gloo and rank 0 alone prints."""
    import json
    out = _run_bench("--gpus", "2", "--launch-check")
    assert out.returncode == 0, out.stderr[-2000:]
    assert "starting 2 ranks" in out.stderr
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d == {"launch_check": True, "world": 2, "ranks_seen": [0, 1], "max_rank": 1.0}


def test_gpus_n_without_cuda_fails_in_the_ranks_after_the_spawn():
    import re
    import torch
    if torch.cuda.is_available():
        import pytest
        pytest.skip("a CUDA device is present: the ranks would run the bench")
    out = _run_bench("--gpus", "2", "--steps", "1")
    assert out.returncode != 0
    assert "starting 2 ranks" in out.stderr
    # the refusal comes from a rank of the spawned pair, not from the parent (the launcher ends the other rank as soon
    # as the first one has failed, so not every rank gets to say it; that both ranks start and meet is what
    # test_gpus_n_starts_its_own_ranks above asserts)
    assert re.search(r"bench\.py \(rank [01] of 2\) needs a CUDA device", out.stderr)
    assert "no CPU fallback" in out.stderr
    assert not [l for l in out.stdout.splitlines() if l.startswith("{")]


def test_launcher_command_is_one_rank_per_gpu_on_loopback():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(["--gpus", "4", "--steps", "2"], 4, port=29999)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29999"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")
