"""The N>1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job value.

The path itself has no cross-GPU exchange (the ranks of the method are emulated inside one GPU), so more GPUs
mean independent replicas; what the processes share is only the barrier and the reduction of the step time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    ms = [4.0, 5.5][rank]                       # rank 1 is the slow one
    worst = bench.max_over_ranks(ms)
    assert worst == 5.5, worst
    v = bench.job_value(dist.get_world_size(), 4.398e12, worst)
    assert abs(v - 2 * 4.398e12 / 5.5e-3 / 1e12) < 1e-9
    dist.barrier()
    if rank == 0:
        print("OK", worst, v)
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
                          "--master-port", "29653", str(script)], capture_output=True, text=True, timeout=240,
                         env={**os.environ, "OMP_NUM_THREADS": "1"})
    assert out.returncode == 0, out.stderr[-2000:]
    assert "OK 5.5" in out.stdout


def test_reference_arm_runs_on_rank_zero_only():
    env = {**os.environ, "RANK": "1", "WORLD_SIZE": "2"}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""      # other ranks exit 0 without work


def test_single_process_value_is_unchanged():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25) == 3.25
    assert abs(bench.job_value(1, 2e12, 2.0) - 1000.0) < 1e-9      # 2 TFLOP in 2 ms
