"""The benchmark's N > 1 path on CPU: two gloo ranks as independent replicas -- the step time is the
slowest rank's, the value counts both ranks' bytes; and the reference arm prints one line on rank 0 only."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 100.0 if rank == 0 else 140.0                  # rank 1 is the slow replica
    ms_step, value = bench.replica_aggregate(ms_local, 10, 7_000_000_000, world, "cpu")
    out[rank] = (ms_step, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_bytes():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank, args=(2, 29517, out), nprocs=2, join=True)
    for rank in (0, 1):
        ms_step, value = out[rank]
        assert ms_step == 14.0                                # max over ranks / steps
        assert abs(value - 2 * 7.0 / 14.0e-3) < 1e-6          # GB/s: both replicas' bytes over the slowest time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.replica_aggregate(50.0, 5, 1_000_000_000, 1, "cpu") == (10.0, 100.0)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c2", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c2", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
