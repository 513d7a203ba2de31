"""Host logic of the benchmark that needs no GPU: the N>1 rank reduction (gloo, world size 2),
the reference arm's output line, and the clock-sample parser."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
    red = bench.max_over_ranks(ms)
    q.put((rank, red, bench.whole_job_tflops(2e12, world, red[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_gloo_world2():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, val in out:
        assert red == [15.0, 3.0]                               # slowest rank decides each timing
        assert val == pytest.approx(2 * 2e12 / 15e-3 / 1e12)    # two replicas' work over that time


def test_single_process_reduction_is_identity():
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_clock_sampler_parses_reasons():
    s = bench.ClockSampler(0)
    s.proc = object()                  # stands for a running nvidia-smi; the lines are given instead of read
    s.lines = ["1965, 1965, 480.1, Not Active, Not Active, Not Active, Not Active",
               "1320, 1965, 998.0, Not Active, Not Active, Not Active, Active",
               "1350, 1965, 990.0, Not Active, Not Active, Not Active, Active"]
    c = s.stop()
    assert c["sm_mhz"] == 1350.0 and c["sm_max_mhz"] == 1965.0 and c["reasons"] == ["sw_power_cap"]


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    # other ranks stay silent
    out1 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                           "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=dict(os.environ, RANK="1"), timeout=60)
    assert out1.returncode == 0 and out1.stdout.strip() == ""


def test_gpus_flag_starts_the_ranks_itself_gloo_world2():
    """`bench.py --gpus 2` without torchrun: the launcher starts two ranks (rendezvous on 127.0.0.1); here they are gloo ranks
    on CPU running a stand-in step, and rank 0's line must report both."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-launch"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["ms_per_rank"] == [10.0, 15.0] and line["ms_per_step"] == 15.0
    assert line["config"]["parallelism"] == "replicas only"


def test_gpus_flag_fails_loudly_when_the_machine_has_fewer_gpus():
    import torch
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(max(have, 1) + 1), "--steps", "1"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode != 0 and out.stdout.strip() == ""
    assert "refusing to report fewer replicas" in out.stderr


def test_leg_selection():
    ns = lambda **kw: type("A", (), dict(dict(legs=None, workload="wan14b_720p", heads=None, density=None,
                                               exact_builder=False, regions=False), **kw))()
    assert bench.legs_from_args(ns()) == set(bench.ALL_LEGS)                    # default run carries every leg
    assert bench.legs_from_args(ns(heads=4)) == set()                           # profiling slices stay lean
    assert bench.legs_from_args(ns(legs="none", regions=True)) == {"regions"}
    assert bench.legs_from_args(ns(legs="configs,density_sweep")) == {"configs", "density_sweep"}
    with pytest.raises(SystemExit):
        bench.legs_from_args(ns(legs="bogus"))
    assert bench.mufu_bound_ms(148 * 16, 128, 1000.0) == pytest.approx(16 * 1024 / 1e9 * 1e3)   # 16 tiles per SM, 1024 clocks each
