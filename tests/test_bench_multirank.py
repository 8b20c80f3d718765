"""Host-side logic of the multi-rank bench path, on CPU with the gloo backend (world size 2).

The operator has no exchange step, so with N GPUs every rank runs an independent replica; the only
cross-rank traffic is the barrier and the max-over-ranks of the timing."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench.barrier()
    slowest = bench.max_over_ranks(10.0 + rank, torch.device("cpu"))
    assert bench.dist_env() == (rank, 0, world)
    out.put((rank, slowest))
    dist.destroy_process_group()


def test_max_over_ranks_and_barrier_with_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results == {0: 11.0, 1: 11.0}          # every rank sees the slowest rank's time


def test_without_a_process_group_the_helpers_are_identities():
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    bench.barrier()


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "3"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_sampled_flops_counts_visible_keys():
    import bench
    from paper_2609_33586_b200.inputs import Workload
    wl = Workload("w", 2, 4, 2, 8, 8, 16, True, "bf16", 0)
    assert bench.sampled_flops(wl, range(8)) == wl.flops + 4.0 * 2 * 4 * 16 * 8 / 2   # sum(i+1) = S(S+1)/2
    nc = wl.with_(causal=False)
    assert bench.sampled_flops(nc, [0, 3]) == 4.0 * 2 * 4 * 16 * 8 * 2
