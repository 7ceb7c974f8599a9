"""The N > 1 path of the benchmark harness on CPU: two gloo ranks.  Blocks are independent, so
ranks share no data-path collective; what has to be right is the bookkeeping around them:
one workload per rank with its own seed, the maximum over ranks as the reported time, the
whole-job token count, and a reference arm that only rank 0 runs."""
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w = bench.make_workload("tiny", seed_offset=rank)
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
    dist.barrier()
    out.put((rank, w.seed, w.block_lens.tolist(), slowest, bench.whole_job_tokens(w, world)))
    dist.destroy_process_group()


def test_two_gloo_ranks_seed_max_and_tokens():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, lens0, max0, tok0), (r1, seed1, lens1, max1, tok1) = res
    assert (r0, r1) == (0, 1)
    assert seed0 != seed1 and lens0 == lens1          # same shape, different draws
    assert max0 == max1 == 15.0                        # the slowest rank's time on every rank
    assert tok0 == tok1 == 2 * 4 * 16                  # 2 ranks x 4 blocks x 16 summary tokens


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5


def test_gpus_flag_means_that_many_ranks():
    sys.path.insert(0, ROOT)
    import bench
    # started by a launcher: --gpus must agree with it
    assert bench.rank_layout(2, {"WORLD_SIZE": "2", "RANK": "1", "LOCAL_RANK": "1"}) == ("run", 1, 2, 1)
    with pytest.raises(SystemExit):
        bench.rank_layout(8, {"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    with pytest.raises(SystemExit):
        bench.rank_layout(1, {"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    # started bare: one GPU runs in place, more GPUs start one rank each through torch's launcher
    assert bench.rank_layout(1, {}) == ("run", 0, 1, 0)
    kind, argv = bench.rank_layout(4, {})
    assert kind == "spawn" and "--nproc-per-node=4" in argv and "127.0.0.1" in argv
    assert argv[argv.index("-m") + 1] == "torch.distributed.run"
    # the reference arm is rank 0's host cores whatever --gpus says
    assert bench.rank_layout(8, {}, impl="reference") == ("run", 0, 1, 0)


def test_bare_launch_with_a_mismatching_world_size_fails_loudly():
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--config", "tiny"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode != 0 and "WORLD_SIZE" in (r.stderr + r.stdout)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
           "--gpus", "2", "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
