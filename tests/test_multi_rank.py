"""The N > 1 path of bench.py on CPU: two gloo ranks.  Ranks run independent replicas (no exchange
on the data path); what they share is the barrier and the max-over-ranks timing."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    from paper_2601_10155_b200 import synth
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w = synth.small_workload(B=2, n_q_heads=4, n_kv_heads=2, L=64)
    mine = bench.rank_workload(w, rank)
    elapsed = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
    dist.barrier()
    reduced = bench.max_over_ranks(elapsed, "cpu")
    seeds = [None] * world
    dist.all_gather_object(seeds, mine.seed)
    out[rank] = (reduced, seeds, bench.job_value(w, world, reduced[0]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_distinct_inputs():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        reduced, seeds, value = res[rank]
        assert reduced == [15.0, 3.0]
        assert len(set(seeds)) == world
        # whole-job value: both replicas' pairs over the slowest rank's time
        assert value == 2 * 4 * 64 * world / (15.0 * 1e-3)


def test_without_a_process_group_the_reduction_is_the_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
