"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path collective).
Checks the max-over-ranks timing, the whole-job aggregate and that only rank 0 reports."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    dist.barrier()
    slowest = bench.max_over_ranks(my_ms)
    value = bench.whole_job_value(world, units_per_rank_per_step=1000, steps=4, max_ms=slowest)
    out[rank] = (slowest, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregate_gloo():
    world, port = 2, 29741
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                        # every rank agrees on the slowest time
    slowest, value = res[0]
    assert slowest == 15.0
    assert value == 2 * 1000 * 4 / 15.0e-3         # units of ALL ranks over the slowest rank's time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(1, 10, 2, 4.0) == 5000.0


def test_reference_arm_prints_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--d", "2048"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--d", "2048"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["metric"] == "node_param_updates_per_sec" and line["higher_is_better"] is True


def test_bytes_per_update_table():
    sys.path.insert(0, ROOT)
    import bench
    from paper_1811_10792_b200 import inputs
    W = inputs.WORKLOADS
    assert bench.bytes_per_update(W["resnet50"]) == 24
    assert bench.bytes_per_update(W["resnet50"], write_z=False) == 20
    assert bench.bytes_per_update(W["transformer"]) == 16
    assert bench.bytes_per_update(W["resnet50_osgp1"]) == 32
