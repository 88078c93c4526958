"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The exchange does not
shard (one GPU holds all P ranks), so N GPUs run N independent replicas; what the
ranks share is only the timing: the max over ranks, and the whole-job throughput."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 * (rank + 1)                      # rank 1 is the slow replica
    slowest = bench.max_over_ranks(ms, dist)
    dist.barrier()
    out[rank] = (slowest, bench.job_throughput(1_000_000_000, world, slowest))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_replica():
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(2, 29631, out), nprocs=2, join=True)
        assert out[0] == out[1]
        slowest, value = out[0]
        assert slowest == 20.0
        assert abs(value - 2 * 1.0 / 0.020) < 1e-9   # 2 replicas x 1 GB in 20 ms = 100 GB/s


def test_single_process_is_its_own_maximum():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.job_throughput(2_000_000_000, 1, 1000.0) == 2.0


def test_reference_arm_runs_on_rank_zero_only():
    """Under torchrun the oracle-timing arm prints one line from rank 0; other ranks exit 0 silently."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "c1", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "c1", "--steps", "2", "--warmup", "1", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
