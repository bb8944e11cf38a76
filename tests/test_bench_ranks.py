"""bench.py with --gpus N > 1 runs N independent replicas; the host-side part of that path
(max of the ranks' times, whole-job value, rank 0 reports) is exercised here with two gloo
ranks on CPU.  Also: the reference arm prints one JSON line with the contract's keys."""
import json
import os
import subprocess
import sys

import pytest

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, device="cpu")     # rank 1 is the slow one
    value = bench.whole_job_value(1000, 4, world, ms)
    out.put((rank, ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 15.0
        assert value == 2 * 1000 * 4 / 15e-3


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, device="cpu") == 3.5
    assert bench.whole_job_value(10, 2, 1, 4.0) == 10 * 2 / 4e-3


def test_reference_arm_prints_contract_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "lstm_small", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "lstm_small", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "elements/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
    assert line["config"]["workload"] == "lstm_small"
    assert line["config"]["sample"].startswith("2 of the workload's 4 simulated workers")


def test_traffic_table_and_gradient_pool_size():
    """roofline.traffic comes from the committed table of ncu captures (keyed by workload and
    kernel, None where nothing was captured); the gradient pool has the workload's iteration
    count."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_1712_01887_b200 import inputs as I
    t = bench._ncu_traffic("resnet50", "k_update_emit")
    assert t is not None and 0.5 < t / (20.0 * 25557032) < 1.5
    assert bench._ncu_traffic("resnet50", "no_such_kernel") is None
    assert bench._ncu_traffic("cfg1", "k_update_emit") is None
    assert bench._pool_size(I.workload("resnet50")) == 10
    assert bench._pool_size(I.workload("lstm")) == 10
    assert bench._pool_size(I.workload("cfg1")) == 5


@pytest.mark.gpu
@pytest.mark.parametrize("flags", [[], ["--graph", "--timeline"], ["--flush-l2", "--no-batch"],
                                   ["--separate-receive", "--timeline"]])
def test_bench_options_print_the_contract_line(flags):
    """The benchmark's own arm on the small L2-resident case with its optional modes: one JSON
    line with the contract's keys, launches counted, a roofline object, and the timeline when
    asked for."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cmd = [sys.executable, os.path.join(root, "bench.py"), "--workload", "cfg1", "--steps", "4",
           "--warmup", "3", "--no-e2e", "--no-cpu-baseline"] + flags
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "dtype", "data", "config", "roofline",
                "gpu_launches", "clocks"):
        assert key in line, key
    assert line["steps"] == 4 and line["value"] > 0 and line["gpu_launches"] > 0
    assert line["roofline"]["bound"] == "hbm" and 0 < line["roofline"]["frac"] < 2
    if "--timeline" in flags:
        tl = line["timeline"]["first_last_block_start"]
        assert len(tl) == line["config"]["simulated_workers"] and len(tl[0]) == 4
        for w in tl:
            assert w[0][0] <= w[1][0] <= w[2][0] <= w[3][0]
    else:
        assert line["timeline"] is None
