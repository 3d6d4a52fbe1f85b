"""The multi-rank paths on CPU ranks (gloo, world size 2).

The benchmark's ranks are independent replicas: their only exchange is the aggregation of the
per-rank figures (maximum of the step times, sums of the work), and the seeds must give every
rank its own shard.  Data-distributed training (Sec. 7.3) exchanges integers only: here the
exchange routine the library's callback uses is run over gloo on what two ranks would hold --
histograms of row shards add up to the histogram of all rows, the maxima of Eq. 5 as float bits
maximise to the global maximum, and the stochastic-rounding stream of a shard is the slice of the
global one at the shard's row offset."""
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


def _dist_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    import oracle
    from paper_2207_09682_b200 import dist as qdist, synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n, nb = 6001, 16
    data = synth.sweep_bins(n, 5, nb, device="cpu", seed=3).numpy()
    g, h = (t.numpy() for t in synth.sweep_gradients(n, device="cpu", seed=4))
    full = oracle.quantize(g, h, bits=3, seed=9, tree=2)
    lo, hi = (0, 2500) if rank == 0 else (2500, n)
    # Eq. 5's maxima: float bits of non-negative floats order like integers
    mx = torch.tensor([np.float32(np.abs(g[lo:hi]).max()).view(np.int32), np.float32(h[lo:hi].max()).view(np.int32), 0],
                      dtype=torch.int32)
    qdist.allreduce_tensor(mx, qdist.REDUCE_MAX_U32)
    ok_max = (np.int32(mx[0]).view(np.float32) == np.float32(full.gmax) and
              np.int32(mx[1]).view(np.float32) == np.float32(full.hmax))
    # the shard's histogram of the globally quantized gradients, packed like the library's words
    hg, hh = oracle.histogram(data[lo:hi], nb, full.gq[lo:hi], full.hq[lo:hi])
    words = torch.from_numpy(hg * (1 << 32) + hh)
    qdist.allreduce_tensor(words, qdist.REDUCE_SUM_I64)
    fg, fh = oracle.histogram(data, nb, full.gq, full.hq)
    w = words.numpy()
    ok_sum = ((w >> 32) == fg).all() and ((w & 0xFFFFFFFF) == fh).all()
    # stochastic rounding keyed by the global row number
    ug, uh = oracle.sr_uniforms(9, 2, lo, hi - lo)
    fug, fuh = oracle.sr_uniforms(9, 2, 0, n)
    ok_key = (ug == fug[lo:hi]).all() and (uh == fuh[lo:hi]).all()
    dist.barrier()
    out.put((rank, bool(ok_max), bool(ok_sum), bool(ok_key)))
    dist.destroy_process_group()


def test_two_ranks_exchange_integers_exactly():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_dist_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, True, True, True), (1, True, True, True)]
