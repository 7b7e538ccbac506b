"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, each with its own sequence, timed with
a max over ranks.  The data path has no collective (ranks work on independent sequences), so this
covers everything that differs from the single-rank run."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2601_18401_b200 import synth
    w = bench.rank_workload(synth.CONFIGS[1].scaled(seq_len=2048, n_q_heads=4, n_kv_heads=2, planted_spans=2), rank)
    x = synth.make_prefill(w, device="cpu")
    dist.barrier()
    slowest = bench.max_over_ranks(10.0 + rank, dist, "cpu")
    out.put((rank, w.seed, float(x["q"].float().sum()), slowest))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_independent_sequences_and_max_timing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, q0, t0), (r1, s1, q1, t1) = res
    assert (r0, r1) == (0, 1) and s0 != s1 and q0 != q1      # each rank has its own sequence
    assert t0 == t1 == 11.0                                  # both report the slowest rank's time


def test_max_over_ranks_is_identity_without_dist():
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5


def _gather_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2601_18401_b200 import sharded
    # the two exchanges of the sequence-sharded decode step: candidates [B,Hq,k], partial results [B,Hq,D+2]
    cand = torch.full((2, 3, 4), rank, dtype=torch.int32)
    part = torch.full((2, 3, 10), float(rank) + 0.5)
    ga, gp = sharded._gather(cand, None), sharded._gather(part, None)
    out.put((rank, tuple(ga.shape), ga[:, 0, 0, 0].tolist(), tuple(gp.shape), gp[:, 1, 2, 3].tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_decode_exchanges_two_ranks():
    """Rank order and shapes of the two all-gathers of the sequence-sharded decode step (gloo, CPU)."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 30500 + os.getpid() % 1000
    procs = [ctx.Process(target=_gather_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, sa, va, sp, vp in res:
        assert sa == (2, 2, 3, 4) and va == [0, 1]
        assert sp == (2, 2, 3, 10) and vp == [0.5, 1.5]


def test_shard_ranges_tile_the_cache():
    from paper_2601_18401_b200 import sharded
    for cap, world in ((1000, 1), (1000, 3), (1048576 + 5, 8), (7, 8), (64, 64)):
        pos = 0
        for r in range(world):
            lo, ln = sharded.shard_range(cap, r, world)
            assert lo == pos and ln >= 0
            pos += ln
        assert pos == cap
