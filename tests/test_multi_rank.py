"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path shards with no data exchange (independent
chunks per rank); what crosses ranks is the barrier and the max over ranks of the timed region."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2602_08722_b200 import synth
    # rank r is slower: the job time is the slowest rank's on every rank
    mine = 100.0 + 50.0 * rank
    got = bench.max_over_ranks(mine, world)
    # independent problems per rank: different seeds, and for the serving mix different cached lengths
    seed_r, lens = bench.rank_workload(dict(synth.WORKLOADS["serving_mix"]), 7, rank)
    seed_fixed, lens_fixed = bench.rank_workload(dict(synth.WORKLOADS["llama8b_32k"]), 7, rank)
    dist.barrier()
    q.put((rank, got, seed_r, lens, seed_fixed, lens_fixed, bench.job_us_per_chunk(got, 10, world)))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_draw_different_inputs():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, s0, l0, f0, lf0, v0), (r1, t1, s1, l1, f1, lf1, v1) = res
    assert (r0, r1) == (0, 1)
    assert t0 == t1 == 150.0                       # max over ranks, on both
    assert v0 == v1 == 150.0 / (10 * 2)            # all ranks' chunks / the slowest rank's time
    assert s0 != s1 and l0 != l1                   # serving mix: each rank its own sequences
    assert f0 != f1 and lf0 == lf1 == [32768]      # fixed-length workload: same shape, different data


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, 1) == 12.5
    assert bench.job_us_per_chunk(100.0, 10, 1) == 10.0
