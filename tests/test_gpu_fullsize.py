"""Parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times (one context, data resident on the device, the default stream).

Where the CPU oracle finishes in seconds it checks everything (whole histograms, whole trees);
for the largest sweep point it checks sampled features one by one, and the properties that
hold at any size (every feature's bins add up to the leaf totals) are checked on all of them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_09682_b200 import binding, synth

pytestmark = pytest.mark.gpu


def check_tree(model, k, ref):
    got = model.tree(k)
    assert got["num_leaves"] == ref.num_leaves
    for key in ("feature", "bin", "left", "right"):
        assert (got[key] == getattr(ref, key)).all(), (k, key)
    assert (got["gain"].view(np.uint64) == ref.gain.view(np.uint64)).all()
    assert (got["leaf_count"] == ref.leaf_count).all()
    assert np.allclose(got["leaf_value"], ref.leaf_value, rtol=1e-5, atol=0)


def run_config(name, trees, **over):
    wl = synth.CONFIGS[name](device="cuda")
    kw = dict(wl.params, seed=2024, num_trees=trees)
    kw.update(over)
    n = wl.bins.shape[0]
    ctx = binding.Context(binding.make_params(**kw))
    ctx.load_binned(wl.bins, wl.n_bins)
    scores = torch.zeros(n, device="cuda")
    model = ctx.train(wl.labels, scores, 0, trees)
    data, y = wl.bins.cpu().numpy(), wl.labels.cpu().numpy()
    ref_scores = np.zeros(n, np.float32)
    prm = oracle.make_params(**kw)
    for k in range(trees):
        check_tree(model, k, oracle.train_tree(data, wl.n_bins, y, ref_scores, prm, k))
    got = scores.cpu().numpy()
    assert np.allclose(got, ref_scores, rtol=1e-5, atol=1e-7)
    assert (got.view(np.uint32) == ref_scores.view(np.uint32)).all()
    return ctx, wl, data


def test_tiny_config_all_trees():
    run_config("tiny", 10)


def test_tall_config_twenty_trees():
    # any differing score bit re-randomises the next tree's stochastic rounding: twenty chained trees
    run_config("tall", 20)


def test_large_config_three_trees_and_root_histogram():
    ctx, wl, data = run_config("large", 3)
    # the root histogram of the next iteration, whole, against Algorithm 1 on the CPU
    n = data.shape[0]
    g = torch.randn(n, device="cuda", generator=torch.Generator(device="cuda").manual_seed(5))
    info = ctx.quantize_gradients(g, None, tree=7)
    ref = oracle.quantize(g.cpu().numpy(), None, bits=4, seed=2024, tree=7)
    hist = ctx.new_hist()
    ctx.build_histograms(0, hist)
    G, H = binding.unpack_hist(hist)
    og, oh = oracle.histogram(data, wl.n_bins, ref.gq, ref.hq)
    assert (G == og).all() and (H == oh).all()
    assert (G.sum(axis=1) == info["G_total"]).all() and (H.sum(axis=1) == n).all()


def test_wide_config_two_trees():
    run_config("wide", 2)


SWEEP_POINTS = [
    # rows, features, bins, bits, features checked on the CPU (None: all)
    (1_000_000, 28, 16, 2, None),
    (4_000_000, 136, 64, 3, 24),
    (16_000_000, 28, 255, 4, None),
    (1_000_000, 1000, 255, 8, 16),
    (4_000_000, 28, 64, 5, None),
    (16_000_000, 1000, 255, 3, 8),
    (2_000_000, 28, 255, 8, None),      # 32+32 local bins: 74 pairs of CTAs, one pass each
    (3_000_001, 136, 64, 7, 20),        # the same with two tile widths and a ragged tail
]


@pytest.mark.parametrize("n,f,nb,bits,sample", SWEEP_POINTS)
def test_sweep_point_histograms(n, f, nb, bits, sample):
    bins = synth.sweep_bins(n, f, nb, device="cuda")
    g, h = synth.sweep_gradients(n, device="cuda")
    ctx = binding.Context(binding.make_params(bits=bits, seed=77))
    ctx.load_binned(bins, nb)
    info = ctx.quantize_gradients(g, h, tree=1)
    ref = oracle.quantize(g.cpu().numpy(), h.cpu().numpy(), bits=bits, seed=77, tree=1)
    assert info["G_total"] == int(ref.gq.astype(np.int64).sum()) and info["H_total"] == int(ref.hq.astype(np.int64).sum())
    cols = np.arange(f) if sample is None else np.sort(np.random.default_rng(f).choice(f, sample, replace=False))
    cols_t = torch.from_numpy(cols).cuda()
    data = bins[:, cols_t].contiguous().cpu().numpy() if sample is not None else bins.cpu().numpy()
    del bins
    hist = ctx.new_hist()
    rows = synth.subset_rows(n, device="cuda")
    rows_np = rows.cpu().numpy().astype(np.uint32)
    for r, r_np in ((None, None), (rows, rows_np)):
        if r is None:
            ctx.build_histograms(0, hist)
        else:
            ctx.build_histograms_rows(r, hist)
        G, H = binding.unpack_hist(hist)
        og, oh = oracle.histogram(data, nb, ref.gq, ref.hq, r_np)
        assert (G[cols] == og).all() and (H[cols] == oh).all()
        # every feature's bins add up to the totals of the rows that were histogrammed
        sel = slice(None) if r_np is None else r_np
        assert (G.sum(axis=1) == int(ref.gq[sel].astype(np.int64).sum())).all()
        assert (H.sum(axis=1) == int(ref.hq[sel].astype(np.int64).sum())).all()


def test_worst_case_accumulation_at_scale():
    # every row in one bin with the extreme gradient level: a CTA's 16+16-bit columns would
    # overflow several times over without the flushes (4 M rows over at most 148 CTAs)
    n = 4_000_000
    data = torch.zeros((n, 28), dtype=torch.uint8, device="cuda")
    data[:, 5] = 3
    for bits in (3, 4, 5):
        kg, kh = oracle.levels(bits)
        ctx = binding.Context(binding.make_params(bits=bits))
        ctx.load_binned(data, 8)
        ctx.quantize_gradients(torch.full((n,), -1.0, device="cuda"), torch.full((n,), 0.25, device="cuda"))
        hist = ctx.new_hist()
        ctx.build_histograms(0, hist)
        G, H = binding.unpack_hist(hist)
        assert G[0, 0] == -kg * n and H[0, 0] == kh * n and G[5, 3] == -kg * n and H[5, 3] == kh * n and H[5, 0] == 0
        rows = synth.subset_rows(n, device="cuda")
        ctx.build_histograms_rows(rows, hist)
        G, H = binding.unpack_hist(hist)
        m = rows.numel()
        assert G[27, 0] == -kg * m and H[27, 0] == kh * m and G[5, 3] == -kg * m


def test_worst_case_accumulation_constant_hessian():
    # constant hessian: the local bins split their 32 bits unevenly (row count below, gradient sum
    # above); all rows in one bin at the extreme gradient level must still come out exact
    n = 6_000_000
    data = torch.zeros((n, 28), dtype=torch.uint8, device="cuda")
    data[:, 9] = 7
    for bits in (2, 4, 5):
        kg, _ = oracle.levels(bits)
        ctx = binding.Context(binding.make_params(bits=bits, objective=1))
        ctx.load_binned(data, 8)
        for sign in (-1.0, 1.0):
            ctx.quantize_gradients(torch.full((n,), sign, device="cuda"), None)
            hist = ctx.new_hist()
            ctx.build_histograms(0, hist)
            G, H = binding.unpack_hist(hist)
            assert G[0, 0] == sign * kg * n and H[0, 0] == n and G[9, 7] == sign * kg * n and H[9, 7] == n and H[9, 0] == 0
            rows = synth.subset_rows(n, device="cuda")
            ctx.build_histograms_rows(rows, hist)
            G, H = binding.unpack_hist(hist)
            assert G[27, 0] == sign * kg * rows.numel() and H[27, 0] == rows.numel()


def test_worst_case_accumulation_wide_tile():
    # a 128-feature tile with many bins: its CTAs look for words that are about to overflow and
    # move only those to the output; every row in one bin at the extreme levels makes the same
    # words hot at every look
    n = 3_000_000
    data = torch.zeros((n, 160), dtype=torch.uint8, device="cuda")
    data[:, 5] = 199
    data[:, 131] = 77
    data[::2, 64] = 100
    for bits in (3, 5):
        kg, kh = oracle.levels(bits)
        ctx = binding.Context(binding.make_params(bits=bits))
        ctx.load_binned(data, 200)
        for sign in (-1.0, 1.0):
            ctx.quantize_gradients(torch.full((n,), sign, device="cuda"), torch.full((n,), 0.25, device="cuda"))
            hist = ctx.new_hist()
            ctx.build_histograms(0, hist)
            G, H = binding.unpack_hist(hist)
            assert G[0, 0] == sign * kg * n and H[0, 0] == kh * n and H[5, 0] == 0
            assert G[5, 199] == sign * kg * n and H[5, 199] == kh * n
            assert G[131, 77] == sign * kg * n and H[131, 77] == kh * n
            assert H[64, 100] == kh * (n // 2) and H[64, 0] == kh * (n // 2) and G[64, 100] == sign * kg * (n // 2)
            assert (G.sum(axis=1) == sign * kg * n).all() and (H.sum(axis=1) == kh * n).all()
            rows = synth.subset_rows(n, device="cuda")
            ctx.build_histograms_rows(rows, hist)
            G, H = binding.unpack_hist(hist)
            m = rows.numel()
            assert G[159, 0] == sign * kg * m and H[159, 0] == kh * m and G[5, 199] == sign * kg * m
            assert (G.sum(axis=1) == sign * kg * m).all() and (H.sum(axis=1) == kh * m).all()
