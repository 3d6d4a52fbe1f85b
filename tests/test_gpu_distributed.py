"""Data-distributed training (Sec. 7.3) with the ranks of one process on one GPU: every rank is a
context on a row shard, driven by a thread of its own; the exchanges go through the library's
callback to a host-side group that adds the ranks' device buffers up.  The trees and the scores
must be those of a single context on all rows, bit for bit, and those of the CPU oracle."""
import threading

import numpy as np
import pytest
import torch

import oracle
from paper_2207_09682_b200 import binding, dist, synth

pytestmark = pytest.mark.gpu


def train_single(data, y, nb, kw, trees):
    ctx = binding.Context(binding.make_params(**kw))
    ctx.load_binned(torch.from_numpy(data).cuda(), nb)
    scores = torch.zeros(len(y), device="cuda")
    model = ctx.train(torch.from_numpy(y).cuda(), scores, 0, trees)
    return model, scores.cpu().numpy()


def train_sharded(data, y, nb, kw, trees, bounds, refit=True):
    world, n = len(bounds) - 1, len(y)
    group = dist.LocalGroup(world)
    out, errors = [None] * world, []

    def worker(r):
        try:
            lo, hi = bounds[r], bounds[r + 1]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                ctx = binding.Context(binding.make_params(**kw))
                if not refit:
                    ctx.set_option(binding.OPT_LEAF_VALUES, 1)
                ctx.load_binned(torch.from_numpy(np.ascontiguousarray(data[lo:hi])).cuda(), nb)
                ctx.set_distributed(r, world, lo, n, group.reducer(r))
                scores = torch.zeros(hi - lo, device="cuda")
                model = ctx.train(torch.from_numpy(np.ascontiguousarray(y[lo:hi])).cuda(), scores, 0, trees)
                stream.synchronize()
                out[r] = (model, scores.cpu().numpy())
        except Exception as e:      # a failed rank must not leave the others waiting
            errors.append((r, e))
            group.barrier.abort()

    threads = [threading.Thread(target=worker, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors and group.error is None, (errors, group.error)
    assert all(o is not None for o in out)
    return out, group


def same_trees(a, b, trees):
    for k in range(trees):
        x, y = a.tree(k), b.tree(k)
        assert x["num_leaves"] == y["num_leaves"]
        for key in ("feature", "bin", "left", "right", "leaf_count"):
            assert (x[key] == y[key]).all(), (k, key)
        assert (x["gain"].view(np.uint64) == y["gain"].view(np.uint64)).all()
        assert (x["leaf_value"].view(np.uint32) == y["leaf_value"].view(np.uint32)).all()


@pytest.mark.parametrize("name,rows,over,cuts", [
    ("tiny", 24_000, dict(num_trees=3), (0.5,)),                               # two even ranks, logistic, 2 bit
    ("tall", 30_001, dict(num_trees=2, num_leaves=63), (0.2, 0.55, 0.9)),       # four uneven ranks
    ("large", 40_000, dict(num_trees=2, num_leaves=31), (0.4,)),               # constant hessian
    ("tall", 20_000, dict(num_trees=2, num_leaves=31, bits=8), (0.3, 0.7)),     # 32+32 local bins
    ("wide", 12_000, dict(num_trees=1, num_leaves=20), (0.45,)),                # 2000 features: 128-byte rows
])
def test_sharded_ranks_train_the_single_context_trees(name, rows, over, cuts):
    wl = synth.CONFIGS[name](device="cpu", rows=rows)
    kw = dict(wl.params, seed=21)
    kw.update(over)
    trees = kw["num_trees"]
    data, y = wl.bins.numpy(), wl.labels.numpy()
    bounds = [0] + [int(c * rows) for c in cuts] + [rows]
    single, single_scores = train_single(data, y, wl.n_bins, kw, trees)
    out, group = train_sharded(data, y, wl.n_bins, kw, trees, bounds)
    for r, (model, scores) in enumerate(out):
        same_trees(model, single, trees)                                        # every rank holds the same trees
        assert (scores.view(np.uint32) == single_scores[bounds[r]:bounds[r + 1]].view(np.uint32)).all()
    assert group.calls > 4 * trees                                              # the ranks did exchange
    # and the oracle on all rows agrees (first tree: structure and values)
    ref_scores = np.zeros(rows, np.float32)
    ref = oracle.train_tree(data, wl.n_bins, y, ref_scores, oracle.make_params(**kw), 0)
    got = out[0][0].tree(0)
    assert got["num_leaves"] == ref.num_leaves and (got["feature"] == ref.feature).all() and (got["bin"] == ref.bin).all()
    assert (got["leaf_count"] == ref.leaf_count).all()
    assert (got["leaf_value"].view(np.uint32) == ref.leaf_value.view(np.uint32)).all()


def test_sharded_ranks_without_refit_and_with_an_empty_side():
    # leaf values from the (global) quantized sums; a shard sorted by one feature leaves whole
    # leaves without rows on one rank
    wl = synth.tiny(device="cpu", rows=16_000)
    order = np.argsort(wl.bins.numpy()[:, 3], kind="stable")
    data, y = np.ascontiguousarray(wl.bins.numpy()[order]), np.ascontiguousarray(wl.labels.numpy()[order])
    kw = dict(wl.params, seed=5, num_trees=2)
    ctx = binding.Context(binding.make_params(**kw))
    ctx.set_option(binding.OPT_LEAF_VALUES, 1)
    ctx.load_binned(torch.from_numpy(data).cuda(), wl.n_bins)
    s = torch.zeros(16_000, device="cuda")
    single = ctx.train(torch.from_numpy(y).cuda(), s, 0, 2)
    out, _ = train_sharded(data, y, wl.n_bins, kw, 2, [0, 5_000, 16_000], refit=False)
    for r, (model, scores) in enumerate(out):
        same_trees(model, single, 2)
    assert (np.concatenate([o[1] for o in out]).view(np.uint32) == s.cpu().numpy().view(np.uint32)).all()


def test_set_distributed_checks_its_arguments():
    ctx = binding.Context(binding.make_params(bits=8))
    cb = dist.LocalGroup(2).reducer(0)
    for args in ((2, 2, 0, 100), (-1, 2, 0, 100), (0, 2, -5, 100), (0, 2, 0, 0), (0, 2, 0, 1 << 32)):
        with pytest.raises(binding.QgbdtError) as e:
            ctx.set_distributed(*args, cb)
        assert e.value.code == binding.ERR_ARG
    with pytest.raises(binding.QgbdtError) as e:
        ctx.set_distributed(0, 2, 0, 30_000_000, cb)      # 3e7 rows * 127 levels: the gradient field overflows
    assert e.value.code == binding.ERR_OVERFLOW
    ctx.set_distributed(0, 1, 0, 0, None)                 # off


def test_nccl_reducer_on_a_group_of_one():
    # the callback the benchmark's sharded mode installs: an NCCL all-reduce on the library's own
    # buffer and stream.  One GPU gives a group of one rank, where the exchange leaves the words as
    # they are; what is checked is the wrapping of pointer, word type and stream.
    import os
    import torch.distributed as tdist
    port = 33500 + os.getpid() % 2000
    tdist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                             device_id=torch.device("cuda", 0))
    try:
        red = dist.TorchDistReducer()
        stream = torch.cuda.Stream()
        words = torch.arange(-5, 1000, dtype=torch.int64, device="cuda") * (1 << 33)
        bits = torch.tensor([0x3F800000, 0x3E800000, 1], dtype=torch.int32, device="cuda")
        stream.wait_stream(torch.cuda.current_stream())
        assert red.callback(None, words.data_ptr(), words.numel(), dist.REDUCE_SUM_I64, stream.cuda_stream) == 0
        assert red.callback(None, bits.data_ptr(), 3, dist.REDUCE_MAX_U32, stream.cuda_stream) == 0
        stream.synchronize()
        assert torch.equal(words, torch.arange(-5, 1000, dtype=torch.int64, device="cuda") * (1 << 33))
        assert bits.tolist() == [0x3F800000, 0x3E800000, 1] and red.calls == 2 and red.words == words.numel() + 3
    finally:
        tdist.destroy_process_group()
