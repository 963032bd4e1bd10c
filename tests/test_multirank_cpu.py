"""Host-side multi-rank logic of the benchmark on CPU (gloo, world size 2): the replicas'
times are combined as the maximum over ranks, and the reference arm works on rank 0 only."""
import os
import subprocess
import sys
from pathlib import Path

import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, str(ROOT))
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 10.0 - rank, 5.0]
    got = bench.slowest_rank(mine, dist, "cpu")
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_slowest_rank_is_elementwise_max_over_two_gloo_ranks():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    assert out[0] == out[1] == [2.0, 10.0, 5.0]


def test_single_process_passthrough():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.slowest_rank([3.0, 4.0], None, "cpu") == [3.0, 4.0]


def test_reference_arm_is_silent_on_nonzero_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
