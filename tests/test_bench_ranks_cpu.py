"""Host-side logic of `bench.py --gpus N`: N independent replicas, no data-path collective.
Run here as two gloo ranks on CPU: the step time is the max over ranks, the value is the
sum of the replicas' tokens over that time, and only rank 0 of the reference arm prints."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")        # rank 1 is the slow one
    out[rank] = (ms, bench.whole_job_value(world, 1000, ms / 10))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_two_gloo_ranks():
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
        assert out[0] == out[1]
        ms, value = out[0]
    assert ms == 15.0
    assert abs(value - 2 * 1000 / 1.5e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, None, "cpu") == 3.25
    assert bench.whole_job_value(1, 16384, 0.5) == 16384 / 0.5e-3


def test_reference_arm_other_ranks_print_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
