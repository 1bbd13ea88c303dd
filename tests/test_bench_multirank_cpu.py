"""Host-side logic of the multi-GPU benchmark path (N independent replicas, no data-path collective), run as two
gloo ranks on the CPU: the job's time is the slowest rank's, the job's throughput counts every rank's work, and
the reference arm leaves all work to rank 0."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r measured (10 + r) ms for the timed region and (30 - 5 r) ms per end-to-end step
        total_ms, e2e_ms = bench.max_over_ranks([10.0 + rank, 30.0 - 5.0 * rank], dist, torch.device("cpu"))
        dist.barrier()
        if rank == 0:
            with open(out, "w") as fh:
                json.dump({"total_ms": total_ms, "e2e_ms": e2e_ms,
                           "value": bench.job_throughput(world, 2.0e12, total_ms / 5)}, fh)
    finally:
        dist.destroy_process_group()


def test_slowest_rank_sets_the_time_and_every_rank_counts(tmp_path):
    out = str(tmp_path / "r0.json")
    mp.spawn(_rank_main, args=(2, 29731, out), nprocs=2, join=True)
    got = json.load(open(out))
    assert got["total_ms"] == 11.0 and got["e2e_ms"] == 30.0
    # 2 ranks x 2 TFLOP per step, 5 steps in 11 ms
    assert abs(got["value"] - 2 * 2.0 / (11.0 / 5 * 1e-3)) < 1e-6


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], None, None) == [3.0, 4.0]
    assert bench.job_throughput(1, 1.0e12, 1000.0) == 1.0


def test_reference_arm_runs_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
