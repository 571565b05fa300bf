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


def test_both_arms_name_the_workload_the_same_way():
    """`config` is a function of the workload and the replica count only (the measured cache
    bytes live beside it, not inside), so the two arms of one run print equal configs."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2503_01586_b200 import inputs as gen
    a = bench.config_of(gen.LLAMA7B_75, 1)
    assert a == bench.config_of(gen.LLAMA7B_75, 1) and a["workload"] == "7b-75pct-b16-ctx4096"
    assert "cache_bytes_per_step" not in a


def _run_bench(*argv, env=None):
    import json
    import subprocess
    e = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], env=e,
                       capture_output=True, text=True, timeout=300)
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    return r.returncode, [json.loads(l) for l in lines], r.stderr


def test_gpus_flag_starts_one_replica_per_rank_by_itself():
    """`bench.py --gpus 2` without torchrun: the script starts its own two ranks (gloo here, no
    GPU), the slowest rank's time decides, the value counts both replicas and exactly one JSON
    line comes out, saying n_gpus 2."""
    code, lines, err = _run_bench("--gpus", "2", "--dry-run-ranks")
    assert code == 0, err
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 2.0
    assert lines[0]["value"] == 2 * 16 / 2.0e-3


def test_gpus_flag_must_agree_with_the_launcher_environment():
    """Under a launcher that already set WORLD_SIZE the flag must say the same number."""
    code, lines, err = _run_bench("--gpus", "4", "--dry-run-ranks",
                                  env={"WORLD_SIZE": "1", "RANK": "0", "LOCAL_RANK": "0"})
    assert code != 0 and not lines and "WORLD_SIZE" in err


def test_gpus_flag_fails_loudly_without_enough_devices():
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        return
    code, lines, err = _run_bench("--gpus", "2", "--steps", "1", "--warmup", "1", "--no-sweep")
    assert code != 0 and not lines and "CUDA device" in err
