"""The N > 1 path of bench.py is "replicas only": no data-path collective, just the max over ranks
of the step time and the summed throughput.  Exercised here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")      # rank 1 is the slow replica
    dist.barrier()
    out[rank] = (ms, bench.aggregate_value(2e12, ms, world))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_two_gloo_ranks():
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
        assert out[0] == out[1]
        ms, value = out[0]
        assert ms == 15.0                                   # the slowest replica sets the time
        assert abs(value - 2 * 2e12 / 15e-3 / 1e12) < 1e-9   # both replicas' work counts


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(1e12, 1.0, 1) == 1000.0


def test_reference_arm_prints_on_rank_zero_only():
    """`--impl reference` under a 2-rank launch: rank 1 exits 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
