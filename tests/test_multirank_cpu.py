"""The N > 1 path of the benchmark on CPU: images are independent, so N GPUs run N replicas with
no data-path collective. What ranks share is the timing protocol (barrier, MAX over ranks of the
device time, whole-job throughput, rank 0 alone prints) and, for the reference arm, that only
rank 0 works. Run here as two gloo processes on 127.0.0.1."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    dist.barrier()
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    total = bench.max_over_ranks(local_ms, dist, "cpu")
    value = bench.replica_throughput(world, 4, total)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"total": total, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_replica_throughput_two_gloo_ranks(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0 == r1                                   # every rank ends with the same numbers
    assert r0["total"] == 15.0                        # the slowest rank's time
    assert abs(r0["value"] - 2 * 4 / 15e-3) < 1e-9    # whole-job images per second


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, None, "cpu") == 7.5
    assert bench.replica_throughput(1, 4, 50.0) == 80.0


def test_reference_arm_only_rank0_works():
    """Under a multi-rank launch the reference arm runs on rank 0; the others exit 0 silently."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
