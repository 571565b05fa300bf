"""The N>1 path of the benchmark is "independent replicas, no data-path collective": the only
cross-rank step is the max over ranks of the timings.  Exercised here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 2.0 - rank, 5.0]
    got = bench.max_over_ranks(dist, mine, "cpu")
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_timings_are_reduced_with_max_over_two_gloo_ranks():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29613, out), nprocs=2, join=True)
    assert out[0] == out[1] == [11.0, 2.0, 5.0]


def test_aggregate_value_counts_every_replica():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_value(1, 16, 0.5) == 32000.0
    assert bench.aggregate_value(8, 16, 0.5) == 8 * 32000.0


def test_reference_arm_config_matches_the_gpu_arm():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2503_01586_b200 import inputs as gen
    a = bench.config_of(gen.LLAMA7B_75, 1)
    b = bench.config_of(gen.LLAMA7B_75, 1, cache_bytes=123)
    b.pop("cache_bytes_per_step")
    assert a == b and a["workload"] == "7b-75pct-b16-ctx4096"
