"""The multi-GPU leg of bench.py is N independent replicas; its only cross-rank logic is the barrier,
the max over ranks and the per-rank seeds.  Covered here with two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from synth import SynthInputs, get_workload
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, True, "cpu")         # rank 1 is the slow one
    wl = bench.replica_workload(get_workload("tiny"), rank, world)
    g = SynthInputs(wl)
    q = g.queries([0])
    res = {"ms": ms, "seed": wl.seed, "qsum": float(q.double().sum()),
           "value": bench.job_value(16, 2, world, ms)}
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump(res, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_use_different_seeds(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.load(open(tmp_path / f"r{r}.json")) for r in (0, 1))
    assert r0["ms"] == r1["ms"] == 15.0
    assert r0["seed"] != r1["seed"] and r0["qsum"] != r1["qsum"]
    assert r0["value"] == r1["value"] == 2 * 16 * 2 / 15.0e-3      # whole-job tokens/s over the slowest rank


def test_single_rank_helpers():
    import bench
    from synth import get_workload
    wl = get_workload("tiny")
    assert bench.replica_workload(wl, 0, 1) is wl
    assert bench.max_over_ranks(3.5, False, "cpu") == 3.5


def test_reference_arm_prints_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
