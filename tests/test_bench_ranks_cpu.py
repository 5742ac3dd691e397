"""The N > 1 leg of bench.py on CPU: two gloo ranks, replicas only -- the job's time is the slowest rank's,
its throughput all ranks' tokens over that time, and only rank 0 of the reference arm prints.  `bench.py --gpus 2`
started by hand launches its own two ranks; without a GPU the CUDA arm refuses loudly instead of falling back."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    out.put((rank, ms, bench.whole_job_tokens_per_s(128, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 15.0
        assert abs(value - 2 * 128 / 15e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_tokens_per_s(128, 1, 64.0) == 2000.0


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def _run_bench(*argv, timeout=600):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], env=env, capture_output=True,
                          text=True, timeout=timeout)


def test_gpus_2_started_by_hand_launches_two_ranks_and_prints_one_line():
    """main() itself: --gpus 2 with no launcher around it re-executes under torch's launcher; the reference arm's
    rank 0 prints the one JSON line (n_gpus 2, the whole 128-token decode), rank 1 exits 0 without work."""
    r = _run_bench("--gpus", "2", "--impl", "reference", "--steps", "1", "--warmup", "0")
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["steps"] == 1
    assert "decode 128 tokens" in line["config"]["workload"] and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["value"] == line["value"] and line["gpu_launches"] == 0


def test_cuda_arm_refuses_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        import pytest
        pytest.skip("a GPU is present")
    for argv in (("--steps", "1", "--warmup", "0"), ("--gpus", "2", "--steps", "1", "--warmup", "0")):
        r = _run_bench(*argv)
        assert r.returncode != 0
        assert "needs a GPU" in (r.stderr + r.stdout)
        assert not [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
