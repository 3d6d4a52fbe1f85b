"""The multi-GPU path of the benchmark on CPU ranks (gloo, world size 2): ranks are independent
replicas, so the only exchange is the aggregation of the per-rank figures -- maximum of the step
times, sums of the work -- and the seeds must give every rank its own shard."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2207_09682_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.tiny(device="cpu", rows=2000, seed=synth.MASTER_SEED + 100 + rank)
    ms, rf, launches = bench.aggregate_ranks(10.0 + rank, 1000.0 * (rank + 1), 7 + rank, dist, "cpu")
    dist.barrier()
    out.put((rank, ms, rf, launches, int(wl.bins.sum()), int(wl.labels.sum())))
    dist.destroy_process_group()


def test_two_ranks_aggregate_and_use_different_shards():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, rf, launches, _, _ in res:
        assert ms == 11.0 and rf == 3000.0 and launches == 15.0      # max of times, sums of work
    assert res[0][4:] != res[1][4:]                                      # the two shards differ


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_ranks(3.5, 10, 4) == (3.5, 10.0, 4.0)
