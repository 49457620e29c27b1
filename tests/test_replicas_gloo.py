"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only, timing meets by a max."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_1611_05402_b200 import replicas
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow one
        value, ms = replicas.whole_job_value(1000, local_ms, torch.device("cpu"))
        dist.barrier()
        with open(f"{out}.{rank}", "w") as f:
            json.dump({"value": value, "ms": ms}, f)
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_all_units_over_the_slowest_rank(tmp_path):
    out = str(tmp_path / "r")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    for rank in range(2):
        with open(f"{out}.{rank}") as f:
            r = json.load(f)
        assert r["ms"] == 25.0
        assert abs(r["value"] - 2 * 1000 / 25e-3) < 1e-6


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    from paper_1611_05402_b200 import replicas
    value, ms = replicas.whole_job_value(500, 4.0, torch.device("cpu"))
    assert ms == 4.0 and value == 500 / 4e-3


def test_reference_arm_leaves_other_ranks_idle():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
