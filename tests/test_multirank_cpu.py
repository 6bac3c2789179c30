"""The N > 1 path of bench.py on CPU (gloo, two ranks): replicas share nothing but the timing
reduction, and only rank 0 of the reference arm reports."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    # every rank timed its own replica: rank r took (1 + r) ms per step and (10 - r) ms end to end
    got = bench.max_over_ranks([1.0 + rank, 10.0 - rank])
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump(got, f)
    dist.destroy_process_group()


def test_timings_are_reduced_by_maximum_over_two_gloo_ranks(tmp_path):
    out = str(tmp_path / "max.json")
    mp.spawn(_rank_main, args=(2, 29611, out), nprocs=2, join=True)
    assert json.load(open(out)) == [2.0, 10.0]


def test_without_a_process_group_values_pass_through():
    import bench

    assert bench.max_over_ranks([0.5, 3]) == [0.5, 3.0]


def test_reference_arm_under_two_ranks_prints_one_line():
    env = dict(os.environ, OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29612", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0", "--ref-heads", "1", "--workload", "tiny_f32"]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
