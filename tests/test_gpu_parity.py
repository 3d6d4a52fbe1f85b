"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Integer results (quantized gradients, histograms, partitions, tree structure) must be
bit-exact; leaf values and scores within 1e-5 relative (they are in fact bit-exact as well,
which the tests assert where the arithmetic guarantees it)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_09682_b200 import binding, synth

pytestmark = pytest.mark.gpu


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def logistic_grads(n, seed):
    g, h = synth.sweep_gradients(n, device="cpu", seed=seed)
    return g.numpy(), h.numpy()


def random_bins(n, f, nb, seed, skew=False):
    if skew:
        return synth.sweep_bins(n, f, nb, device="cpu", seed=seed).numpy()
    r = np.random.default_rng(seed)
    return r.integers(0, nb, size=(n, f), dtype=np.uint8)


def make_ctx(data, nb, **kw):
    ctx = binding.Context(binding.make_params(**kw))
    ctx.load_binned(dev(data), nb)
    return ctx


# ------------------------------------------------------------------ gradients and quantizer

@pytest.mark.parametrize("objective", [0, 1])
def test_gradients_bit_exact(objective):
    n = 100_003
    r = np.random.default_rng(1)
    s = (r.normal(size=n) * 5).astype(np.float32)
    s[:7] = [0.0, 40.0, -40.0, 100.0, -100.0, 1e-8, -17.3]
    y = (r.random(n) < 0.5).astype(np.float32) if objective == 0 else r.normal(size=n).astype(np.float32)
    ctx = make_ctx(random_bins(n, 3, 4, 0), 4, objective=objective)
    g = torch.empty(n, device="cuda")
    h = torch.empty(n, device="cuda") if objective == 0 else None
    ctx.compute_gradients(dev(s), dev(y), g, h)
    og, oh = oracle.gradients(objective, s, y)
    assert (g.cpu().numpy().view(np.uint32) == og.view(np.uint32)).all()
    if objective == 0:
        assert (h.cpu().numpy().view(np.uint32) == oh.view(np.uint32)).all()


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("mode,rounding,const_h", [(0, 0, False), (1, 0, False), (0, 1, False), (0, 0, True)])
def test_quantizer_bit_exact(bits, mode, rounding, const_h):
    n = 200_001
    g, h = logistic_grads(n, 10 + bits)
    if const_h:
        h = None
    ctx = make_ctx(random_bins(n, 2, 4, 0), 4, bits=bits, hess_levels_mode=mode, rounding=rounding, seed=0xABCDEF123)
    gq = torch.empty(n, dtype=torch.int8, device="cuda")
    hq = torch.empty(n, dtype=torch.uint8, device="cuda")
    info = ctx.quantize_gradients(dev(g), None if h is None else dev(h), tree=5, gq=gq, hq=hq)
    ref = oracle.quantize(g, h, bits=bits, seed=0xABCDEF123, tree=5, hess_levels_mode=mode, rounding=rounding)
    assert (gq.cpu().numpy() == ref.gq).all()
    assert (hq.cpu().numpy() == ref.hq).all()
    kg, kh = oracle.levels(bits, mode)
    assert info["g_scale"] == ref.gmax / kg
    assert info["h_scale"] == (1.0 if const_h else ref.hmax / kh)
    assert info["G_total"] == int(ref.gq.astype(np.int64).sum())
    assert info["H_total"] == int(ref.hq.astype(np.int64).sum())


def test_quantizer_rejects_bad_values():
    n = 5000
    g, h = logistic_grads(n, 3)
    ctx = make_ctx(random_bins(n, 2, 4, 0), 4, bits=3)
    for bad_g, bad_h in ((np.nan, None), (np.inf, None), (300.0, None), (None, -0.5), (None, np.nan)):
        g2, h2 = g.copy(), h.copy()
        if bad_g is not None:
            g2[1234] = bad_g
        if bad_h is not None:
            h2[4321] = bad_h
        with pytest.raises(binding.QgbdtError) as e:
            ctx.quantize_gradients(dev(g2), dev(h2))
        assert e.value.code == binding.ERR_VALUE
        with pytest.raises(ValueError):
            oracle.quantize(g2, h2, bits=3)
    ctx.quantize_gradients(dev(g), dev(h))     # the context is still usable


# ------------------------------------------------------------------ histograms

HIST_CASES = [
    # rows, features, bins, bits, skew
    (1, 1, 2, 2, False),
    (37, 3, 5, 3, False),
    (5000, 28, 64, 2, False),
    (70_001, 28, 255, 3, False),
    (70_001, 28, 255, 4, True),
    (9_999, 33, 16, 3, True),
    (20_011, 136, 255, 3, True),
    (12_345, 200, 64, 4, False),
    (6_007, 260, 256, 2, True),
    (30_000, 28, 255, 8, True),
    (8_191, 136, 64, 5, False),
    (4_097, 150, 255, 8, False),
    (300_000, 28, 255, 4, False),
    (50_003, 28, 255, 6, False),        # first bit width with 32+32 local bins
    (50_003, 28, 64, 7, True),
    (25_001, 136, 255, 6, True),        # two tile widths, 32+32 local bins
    (25_001, 136, 128, 7, False),
]


@pytest.mark.parametrize("n,f,nb,bits,skew", HIST_CASES)
def test_histogram_bit_exact(n, f, nb, bits, skew):
    data = random_bins(n, f, nb, 100 + f, skew)
    g, h = logistic_grads(n, 200 + bits)
    ctx = make_ctx(data, nb, bits=bits, seed=9)
    ctx.quantize_gradients(dev(g), dev(h), tree=1)
    ref = oracle.quantize(g, h, bits=bits, seed=9, tree=1)
    hist = ctx.new_hist()
    # root leaf: all rows
    ctx.build_histograms(0, hist)
    G, H = binding.unpack_hist(hist)
    og, oh = oracle.histogram(data, nb, ref.gq, ref.hq)
    assert (G == og).all() and (H == oh).all()
    # about half of the rows, ascending (a leaf after one split)
    rows = synth.subset_rows(n, device="cpu", seed=n).numpy().astype(np.uint32)
    ctx.build_histograms_rows(dev(rows.view(np.int32)), hist)
    G, H = binding.unpack_hist(hist)
    og, oh = oracle.histogram(data, nb, ref.gq, ref.hq, rows)
    assert (G == og).all() and (H == oh).all()
    # shuffled rows with repeats, and the empty leaf
    r = np.random.default_rng(5)
    rows = r.integers(0, n, size=max(1, n // 3)).astype(np.uint32)
    ctx.build_histograms_rows(dev(rows.view(np.int32)), hist)
    G, H = binding.unpack_hist(hist)
    og, oh = oracle.histogram(data, nb, ref.gq, ref.hq, rows)
    assert (G == og).all() and (H == oh).all()
    ctx.build_histograms_rows(torch.zeros(0, dtype=torch.int32, device="cuda"), hist)
    assert not hist.any()


def test_histogram_worst_case_accumulation():
    # every row in one bin with the extreme gradient level: exercises the 16+16 flush bound
    for bits, n in ((2, 200_000), (3, 150_000), (4, 150_000)):
        data = np.zeros((n, 28), np.uint8)
        data[:, 5] = 3
        kg, kh = oracle.levels(bits)
        g = np.full(n, -1.0, np.float32)
        h = np.full(n, 0.25, np.float32)
        ctx = make_ctx(data, 8, bits=bits)
        ctx.quantize_gradients(dev(g), dev(h))
        hist = ctx.new_hist()
        ctx.build_histograms(0, hist)
        G, H = binding.unpack_hist(hist)
        assert G[0, 0] == -kg * n and H[0, 0] == kh * n and G[5, 3] == -kg * n and H[5, 0] == 0
        g[:] = 1.0
        ctx.quantize_gradients(dev(g), dev(h))
        ctx.build_histograms(0, hist)
        G, H = binding.unpack_hist(hist)
        assert G[27, 0] == kg * n and H[27, 0] == kh * n


def test_histogram_worst_case_accumulation_other_hessian_levels():
    # hess_levels_mode 1 (2^B - 1 hessian levels): one more level per row, so a column fills up
    # sooner (another flush interval); all rows in one bin at the extreme levels
    for bits, n in ((2, 200_000), (4, 150_000), (5, 120_000)):
        data = np.zeros((n, 28), np.uint8)
        data[:, 11] = 6
        kg, kh = oracle.levels(bits, 1)
        assert kh == (1 << bits) - 1
        g = np.full(n, -1.0, np.float32)
        h = np.full(n, 0.25, np.float32)
        ctx = make_ctx(data, 8, bits=bits, hess_levels_mode=1)
        ctx.quantize_gradients(dev(g), dev(h))
        ref = oracle.quantize(g, h, bits=bits, hess_levels_mode=1)
        hist = ctx.new_hist()
        ctx.build_histograms(0, hist)
        G, H = binding.unpack_hist(hist)
        og, oh = oracle.histogram(data, 8, ref.gq, ref.hq)
        assert (G == og).all() and (H == oh).all()
        assert G[0, 0] == -kg * n and H[0, 0] == kh * n and G[11, 6] == -kg * n and H[11, 0] == 0
        rows = synth.subset_rows(n, device="cpu", seed=3).numpy().astype(np.uint32)
        ctx.build_histograms_rows(dev(rows.view(np.int32)), hist)
        G, H = binding.unpack_hist(hist)
        assert G[27, 0] == -kg * len(rows) and H[27, 0] == kh * len(rows)


def test_row_list_longer_than_the_histogram_word_allows_is_refused():
    # a list may repeat rows: 8-bit gradients, 17 M entries -> 17e6 * 127 > 2^31 - 1
    data = random_bins(1000, 4, 8, 0)
    g, h = logistic_grads(1000, 1)
    ctx = make_ctx(data, 8, bits=8)
    ctx.quantize_gradients(dev(g), dev(h))
    rows = torch.zeros(17_000_000, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.QgbdtError) as e:
        ctx.build_histograms_rows(rows, ctx.new_hist())
    assert e.value.code == binding.ERR_OVERFLOW


def test_histogram_column_major_input_and_constant_hessian():
    n, f, nb = 40_000, 31, 100
    data = random_bins(n, f, nb, 77)
    g, _ = logistic_grads(n, 8)
    ctx = binding.Context(binding.make_params(bits=4, objective=1))
    ctx.load_binned(dev(np.ascontiguousarray(data.T)), nb, layout=1)
    ctx.quantize_gradients(dev(g), None)
    ref = oracle.quantize(g, None, bits=4, seed=1)
    hist = ctx.new_hist()
    ctx.build_histograms(0, hist)
    G, H = binding.unpack_hist(hist)
    og, oh = oracle.histogram(data, nb, ref.gq, ref.hq)
    assert (G == og).all() and (H == oh).all()
    for j in range(f):
        assert (H[j] == np.bincount(data[:, j], minlength=nb)).all()


@pytest.mark.parametrize("n,f,nb,const_h", [(70_001, 28, 255, False), (20_011, 136, 64, False), (9_999, 33, 16, True),
                                            (300_000, 28, 255, True), (5_000, 300, 256, False)])
def test_floating_point_histogram_matches_double_precision_sums(n, f, nb, const_h):
    # Algorithm 1 with the original gradients in single precision (the unquantized baseline): float
    # atomics add in any order, so each sum may differ from the double-precision one by single-precision
    # rounding of its partial sums: at most (terms in the bin) * 2^-23 * (sum of the magnitudes)
    data = random_bins(n, f, nb, 300 + f, skew=True)
    g, h = logistic_grads(n, 17)
    if const_h:
        h = None
    ctx = make_ctx(data, nb, bits=3)
    rows = synth.subset_rows(n, device="cpu", seed=n).numpy().astype(np.uint32)
    for r in (None, rows):
        hist = ctx.build_histograms_fp32(dev(g), None if h is None else dev(h),
                                         None if r is None else dev(r.view(np.int32))).cpu().numpy().astype(np.float64)
        og, oh = oracle.histogram_fp(data, nb, g, h, r)
        ag, _ = oracle.histogram_fp(data, nb, np.abs(g), None, r)       # sum of |g| and row count per bin
        cnt = oracle.histogram_fp(data, nb, np.ones_like(g), None, r)[0]
        tol_g = cnt * 2.0 ** -23 * ag + 1e-6
        tol_h = cnt * 2.0 ** -23 * np.maximum(oh, 1.0) + 1e-6
        assert (np.abs(hist[:, :, 0] - og) <= tol_g).all()
        assert (np.abs(hist[:, :, 1] - oh) <= tol_h).all()
        if const_h:
            assert (hist[:, :, 1] == oh).all()                             # counts below 2^24 are exact in float


def test_histogram_subtraction():
    n, f, nb = 50_000, 40, 64
    data = random_bins(n, f, nb, 1, True)
    g, h = logistic_grads(n, 2)
    ctx = make_ctx(data, nb, bits=3)
    ctx.quantize_gradients(dev(g), dev(h))
    ref = oracle.quantize(g, h, bits=3, seed=1)
    rows = np.arange(n, dtype=np.uint32)
    small, large = rows[data[:, 7] <= 1], rows[data[:, 7] > 1]
    hp, hs, hl = ctx.new_hist(), ctx.new_hist(), ctx.new_hist()
    ctx.build_histograms(0, hp)
    ctx.build_histograms_rows(dev(small.view(np.int32)), hs)
    ctx.subtract_histograms(hp, hs, hl)
    G, H = binding.unpack_hist(hl)
    og, oh = oracle.histogram(data, nb, ref.gq, ref.hq, large)
    assert (G == og).all() and (H == oh).all()
    ctx.subtract_histograms(hp, hs, hp)          # in place
    assert torch.equal(hp, hl)


def test_load_rejects_bad_codes_and_arguments():
    data = random_bins(1000, 5, 10, 0)
    ctx = binding.Context(binding.make_params())
    with pytest.raises(binding.QgbdtError) as e:
        ctx.load_binned(dev(data), 9)
    assert e.value.code == binding.ERR_VALUE
    with pytest.raises(binding.QgbdtError) as e:
        ctx.load_binned(dev(data), 300)
    assert e.value.code == binding.ERR_ARG
    hist = torch.zeros((5, 10), dtype=torch.int64, device="cuda")
    with pytest.raises(binding.QgbdtError) as e:
        ctx.build_histograms(0, hist)
    assert e.value.code == binding.ERR_STATE
    ctx.load_binned(dev(data), 10)
    with pytest.raises(binding.QgbdtError) as e:
        ctx.build_histograms(0, hist)            # not quantized yet
    assert e.value.code == binding.ERR_STATE
    big = binding.Context(binding.make_params(bits=8))
    # 2e9 rows * 127 levels cannot fit the 32-bit gradient field: refused before any allocation
    rc = big.lib.qgbdt_load_binned(big.h, binding._dptr(dev(data)), binding.C.c_int64(2_000_000_000),
                                   binding.C.c_int32(1), binding.C.c_int32(4), binding.C.c_int32(0),
                                   binding.C.c_int64(1), binding._stream())
    assert rc == binding.ERR_OVERFLOW


# ------------------------------------------------------------------ split finding

@pytest.mark.parametrize("n,f,nb,bits,const_h", [(30_000, 28, 64, 2, False), (30_000, 28, 255, 3, False),
                                                 (20_000, 300, 255, 3, False), (30_000, 28, 255, 4, True),
                                                 (5_000, 7, 33, 8, False), (500, 2, 2, 3, False)])
def test_find_best_split_bit_exact(n, f, nb, bits, const_h):
    data = random_bins(n, f, nb, 3, skew=True)
    g, h = logistic_grads(n, 4)
    g = (g + 0.3 * (data[:, f // 2] > nb // 3)).astype(np.float32)      # plant a signal
    if const_h:
        h = None
    kw = dict(bits=bits, objective=1 if const_h else 0, min_data_in_leaf=20, seed=2)
    ctx = make_ctx(data, nb, **kw)
    info = ctx.quantize_gradients(dev(g), None if h is None else dev(h))
    ref = oracle.quantize(g, h, bits=bits, seed=2)
    hist = ctx.new_hist()
    for rows in (None, synth.subset_rows(n, device="cpu", seed=1).numpy().astype(np.uint32)):
        if rows is None:
            ctx.build_histograms(0, hist)
            sel = np.arange(n)
        else:
            ctx.build_histograms_rows(dev(rows.view(np.int32)), hist)
            sel = rows
        G, H = int(ref.gq[sel].astype(np.int64).sum()), int(ref.hq[sel].astype(np.int64).sum())
        got = ctx.find_best_split(hist, G, H, len(sel))
        og, oh = oracle.histogram(data, nb, ref.gq, ref.hq, sel.astype(np.uint32))
        want = oracle.find_split(og, oh, G, H, len(sel), ref.gmax, ref.hmax, const_h, oracle.make_params(**kw))
        assert got.valid == want.valid == 1
        for key in ("feature", "bin", "gl", "hl", "gr", "hr", "nl_est", "nr_est"):
            assert getattr(got, key) == getattr(want, key), key
        assert np.float64(got.gain).view(np.uint64) == np.float64(want.gain).view(np.uint64)


def test_find_best_split_ties_and_invalid():
    # identical features: the lowest feature and lowest bin must win; a leaf below 2*min_data has no split
    n, nb = 4000, 8
    col = np.random.default_rng(0).integers(0, nb, size=n, dtype=np.uint8)
    data = np.stack([col] * 40, axis=1)
    g = np.where(col <= 2, -0.5, 0.5).astype(np.float32)
    h = np.full(n, 0.25, np.float32)
    kw = dict(bits=2, min_data_in_leaf=20)
    ctx = make_ctx(data, nb, **kw)
    ctx.quantize_gradients(dev(g), dev(h))
    ref = oracle.quantize(g, h, bits=2)
    hist = ctx.new_hist()
    ctx.build_histograms(0, hist)
    G, H = int(ref.gq.astype(np.int64).sum()), int(ref.hq.astype(np.int64).sum())
    got = ctx.find_best_split(hist, G, H, n)
    og, oh = oracle.histogram(data, nb, ref.gq, ref.hq)
    want = oracle.find_split(og, oh, G, H, n, ref.gmax, ref.hmax, False, oracle.make_params(**kw))
    assert (got.feature, got.bin) == (want.feature, want.bin) == (0, 2)
    rows = np.arange(30, dtype=np.uint32)
    ctx.build_histograms_rows(dev(rows.view(np.int32)), hist)
    G, H = int(ref.gq[:30].astype(np.int64).sum()), int(ref.hq[:30].astype(np.int64).sum())
    assert ctx.find_best_split(hist, G, H, 30).valid == 0


# ------------------------------------------------------------------ partition

def test_split_leaf_is_the_stable_partition():
    n, f, nb = 123_457, 37, 50
    data = random_bins(n, f, nb, 6, skew=True)
    ctx = make_ctx(data, nb, num_leaves=8)
    leaves = {0: np.arange(n, dtype=np.uint32)}
    plan = [(0, 5, 20), (0, 36, 0), (1, 0, 48), (2, 17, 10), (1, 9, 49), (3, 1, 0)]
    for leaf, feat, thr in plan:
        right, nl, nr = ctx.split_leaf(leaf, feat, thr)
        out, onl = oracle.partition(data, leaves[leaf], feat, thr)
        assert (nl, nr) == (onl, len(out) - onl)
        leaves[leaf], leaves[right] = out[:onl], out[onl:]
        for l in (leaf, right):
            assert (ctx.get_leaf_rows(l).numpy() == leaves[l].astype(np.int64)).all()
    ctx.reset_leaves()
    assert (ctx.get_leaf_rows(0).numpy() == np.arange(n)).all()


# ------------------------------------------------------------------ refit

@pytest.mark.parametrize("const_h", [False, True])
def test_refit_bit_exact(const_h):
    n, f, nb = 80_000, 10, 16
    data = random_bins(n, f, nb, 8)
    g, h = logistic_grads(n, 9)
    if const_h:
        h = None
    kw = dict(num_leaves=6, learning_rate=0.1, lambda_l2=0.5, objective=1 if const_h else 0)
    ctx = make_ctx(data, nb, **kw)
    leaves = {0: np.arange(n, dtype=np.uint32)}
    for leaf, feat, thr in [(0, 1, 7), (1, 2, 3), (0, 3, 12), (2, 4, 1), (3, 5, 0)]:
        right, nl, nr = ctx.split_leaf(leaf, feat, thr)
        out, onl = oracle.partition(data, leaves[leaf], feat, thr)
        leaves[leaf], leaves[right] = out[:onl], out[onl:]
    w, v = ctx.refit_leaves(dev(g), None if h is None else dev(h), n_leaves=6)
    for l in range(6):
        ow, ov = oracle.refit(g, h, leaves[l], lambda_l2=0.5, learning_rate=0.1)
        assert w[l] == ow and v[l] == ov


def test_refit_with_an_empty_leaf_next_to_a_full_one():
    # a user-chosen split that sends every row left makes an empty right leaf at the offset where
    # the next leaf starts; the rows there must still be credited to the leaf that owns them
    n, f, nb = 30_000, 6, 16
    data = random_bins(n, f, nb, 12)
    g, h = logistic_grads(n, 13)
    ctx = make_ctx(data, nb, num_leaves=5, learning_rate=0.3)
    leaves = {0: np.arange(n, dtype=np.uint32)}
    for leaf, feat, thr in [(0, 2, 7), (0, 1, nb - 1), (0, 3, 4)]:     # the second split leaves leaf 2 empty
        right, nl, nr = ctx.split_leaf(leaf, feat, thr)
        out, onl = oracle.partition(data, leaves[leaf], feat, thr)
        assert (nl, nr) == (onl, len(out) - onl)
        leaves[leaf], leaves[right] = out[:onl], out[onl:]
    assert len(leaves[2]) == 0 and len(leaves[1]) > 0
    w, v = ctx.refit_leaves(dev(g), dev(h), n_leaves=4)
    for l in range(4):
        ow, ov = oracle.refit(g, h, leaves[l], learning_rate=0.3)
        assert w[l] == ow and v[l] == ov, l
    # the score update routes every row to its own leaf's value
    scores = torch.zeros(n, device="cuda")
    ctx.apply_leaf_values(scores)
    want = np.zeros(n, np.float32)
    for l in range(4):
        want[leaves[l]] = v[l]
    assert (scores.cpu().numpy() == want).all()


# ------------------------------------------------------------------ training

def compare_trees(model, k, ref):
    got = model.tree(k)
    assert got["num_leaves"] == ref.num_leaves
    for key in ("feature", "bin", "left", "right"):
        assert (got[key] == getattr(ref, key)).all(), (k, key)
    assert (got["gain"].view(np.uint64) == ref.gain.view(np.uint64)).all()
    assert (got["leaf_count"] == ref.leaf_count).all()
    assert np.allclose(got["leaf_value"], ref.leaf_value, rtol=1e-5, atol=0)
    assert (got["leaf_value"].view(np.uint32) == ref.leaf_value.view(np.uint32)).all()


TRAIN_CASES = [
    ("tiny", 20_000, dict(num_trees=4)),
    ("tall", 30_000, dict(num_trees=3, num_leaves=63)),
    ("large", 40_000, dict(num_trees=3, num_leaves=63)),
    ("wide", 3_000, dict(num_trees=2, num_leaves=15)),
    # more than 512 features: per-leaf constants and the best split over the features in kernels of their own
    ("wide600", 9_000, dict(num_trees=2, num_leaves=40)),
    # 32+32 local bins inside tree growth (two passes over the smaller child's rows)
    ("tall", 30_000, dict(num_trees=3, num_leaves=63, bits=8)),
    ("tall", 30_000, dict(num_trees=3, num_leaves=63, bits=6)),
    ("large", 40_000, dict(num_trees=2, num_leaves=31, bits=7)),
    ("tall", 30_000, dict(num_trees=2, num_leaves=31, bits=5, hess_levels_mode=1)),
    ("tiny", 20_000, dict(num_trees=2, rounding=1)),
    # the smallest trees, and the most leaves a context takes (thousands of growth records in the commit step)
    ("tiny", 5_000, dict(num_trees=2, num_leaves=1)),
    ("tiny", 5_000, dict(num_trees=2, num_leaves=2)),
    ("tiny", 5_000, dict(num_trees=2, num_leaves=3)),
    ("tall", 60_000, dict(num_trees=2, num_leaves=4096, min_data_in_leaf=3)),
    ("tall", 40_000, dict(num_trees=1, num_leaves=1500, min_data_in_leaf=1, bits=2)),
]


def train_case(name, rows, over, column_copy=None, refit=True):
    if name.startswith("wide"):
        wl = synth.wide(device="cpu", rows=rows, features=600 if name == "wide600" else 300)
    else:
        wl = synth.CONFIGS[name](device="cpu", rows=rows)
    kw = dict(wl.params, seed=11)
    kw.update(over)
    data, y = wl.bins.numpy(), wl.labels.numpy()
    ctx = binding.Context(binding.make_params(**kw))
    if column_copy is not None:
        ctx.set_option(binding.OPT_COLUMN_COPY, column_copy)
    if not refit:
        ctx.set_option(binding.OPT_LEAF_VALUES, 1)
    ctx.load_binned(dev(data), wl.n_bins)
    scores = torch.zeros(rows, device="cuda")
    model = ctx.train(dev(y), scores, 0, kw["num_trees"])
    ref_scores = np.zeros(rows, np.float32)
    prm = oracle.make_params(**kw)
    for k in range(kw["num_trees"]):
        ref = oracle.train_tree(data, wl.n_bins, y, ref_scores, prm, k, refit=refit)
        compare_trees(model, k, ref)
    got = scores.cpu().numpy()
    assert np.allclose(got, ref_scores, rtol=1e-5, atol=1e-7)
    assert (got.view(np.uint32) == ref_scores.view(np.uint32)).all()
    return ctx


@pytest.mark.parametrize("name,rows,over", [TRAIN_CASES[0], TRAIN_CASES[2], TRAIN_CASES[5]])
def test_training_with_leaf_values_from_the_quantized_sums(name, rows, over):
    # Sec. 4.2 without refitting: w~ from the integer sums of every leaf; trees, values and scores as the oracle's
    train_case(name, rows, over, refit=False)


@pytest.mark.parametrize("name,rows,over", TRAIN_CASES)
def test_training_matches_oracle(name, rows, over):
    train_case(name, rows, over)


def test_training_without_the_column_copy():
    # the row partition reads the split feature from the tiles when there is no column-major copy
    # (its allocation failed, or the option switched it off): same trees, and the context says
    # which path it took
    for name, rows, over in (TRAIN_CASES[1], TRAIN_CASES[3]):
        for want in (0, 1):
            ctx = train_case(name, rows, over, column_copy=want)
            assert ctx.get_info(binding.INFO_COLUMN_COPY) == want
    ctx = binding.Context(binding.make_params())
    with pytest.raises(binding.QgbdtError) as e:
        ctx.set_option(binding.OPT_COLUMN_COPY, 2)
    assert e.value.code == binding.ERR_ARG
    with pytest.raises(binding.QgbdtError) as e:
        ctx.set_option(99, 0)
    assert e.value.code == binding.ERR_ARG


def test_training_resumes_and_host_variant_agrees():
    wl = synth.tiny(device="cpu", rows=15_000)
    kw = dict(wl.params, seed=3, num_trees=4)
    data, y = wl.bins.numpy(), wl.labels.numpy()
    ctx = make_ctx(data, wl.n_bins, **kw)
    s1 = torch.zeros(15_000, device="cuda")
    m_all = ctx.train(dev(y), s1, 0, 4)
    s2 = torch.zeros(15_000, device="cuda")
    ctx.train(dev(y), s2, 0, 2)
    m_tail = ctx.train(dev(y), s2, 2, 2)          # trees 2, 3 from the scores after trees 0, 1
    assert torch.equal(s1, s2)
    for k in range(2):
        a, b = m_all.tree(2 + k), m_tail.tree(k)
        assert all((a[key] == b[key]).all() for key in ("feature", "bin", "left", "right", "leaf_value"))
    ctx_h = binding.Context(binding.make_params(**kw))
    ctx_h.load_binned(wl.bins.contiguous(), wl.n_bins)     # host matrix
    s3 = torch.zeros(15_000)
    m_host = ctx_h.train(wl.labels.contiguous(), s3, 0, 4)  # host labels / scores
    assert torch.equal(s3, s1.cpu())
    assert (m_host.feature == m_all.feature).all() and (m_host.leaf_value == m_all.leaf_value).all()


def test_phase_timers_cover_every_phase_and_do_not_change_the_trees():
    wl = synth.tiny(device="cpu", rows=15_000)
    kw = dict(wl.params, seed=3, num_trees=2)
    data, y = wl.bins.numpy(), wl.labels.numpy()
    ctx = make_ctx(data, wl.n_bins, **kw)
    s1 = torch.zeros(15_000, device="cuda")
    m1 = ctx.train(dev(y), s1, 0, 2)                 # growth replayed from the graph
    ctx.profile_histograms(True)
    s2 = torch.zeros(15_000, device="cuda")
    m2 = ctx.train(dev(y), s2, 0, 2)                 # the same on the stream, every phase timed
    t = ctx.get_timings()
    prof = ctx.get_histogram_profile()
    ctx.profile_histograms(False)
    assert torch.equal(s1, s2) and (m1.feature == m2.feature).all() and (m1.leaf_value == m2.leaf_value).all()
    assert set(t) == set(binding.PHASES)
    for name, v in t.items():
        assert v["intervals"] >= 2 and v["ms"] > 0.0, name
    assert t["root_histogram"]["intervals"] == 2 and t["gradients"]["intervals"] == 2
    hist_ms = t["root_histogram"]["ms"] + t["child_histograms"]["ms"]
    assert abs(prof["total_ms"] - hist_ms) < 1e-6 and prof["builds"] == 2 + int(m2.num_leaves.sum()) - 2


def test_stepwise_calls_compose_to_the_trained_tree():
    wl = synth.tiny(device="cpu", rows=12_000)
    kw = dict(wl.params, seed=5, num_leaves=8, num_trees=1)
    data, y = wl.bins.numpy(), wl.labels.numpy()
    n = 12_000
    ctx = make_ctx(data, wl.n_bins, **kw)
    scores = torch.zeros(n, device="cuda")
    model = ctx.train(dev(y), scores, 0, 1)
    tree = model.tree(0)
    # the same tree by hand: gradients, quantize, then build / find / split by largest gain
    ctx.reset_leaves()
    g, h = torch.empty(n, device="cuda"), torch.empty(n, device="cuda")
    ctx.compute_gradients(torch.zeros(n, device="cuda"), dev(y), g, h)
    info = ctx.quantize_gradients(g, h, tree=0)
    hists = {0: ctx.new_hist()}
    ctx.build_histograms(0, hists[0])
    tot = {0: (info["G_total"], info["H_total"], n)}
    best = {0: ctx.find_best_split(hists[0], *tot[0])}
    for node in range(tree["num_leaves"] - 1):
        pick = max((l for l in best if best[l].valid), key=lambda l: (best[l].gain, -l))
        s = best[pick]
        assert (s.feature, s.bin) == (tree["feature"][node], tree["bin"][node])
        right, nl, nr = ctx.split_leaf(pick, s.feature, s.bin)
        tot[pick], tot[right] = (s.gl, s.hl, nl), (s.gr, s.hr, nr)
        small, large = (pick, right) if nl <= nr else (right, pick)
        parent = hists[pick]
        hists[small] = ctx.new_hist()
        ctx.build_histograms(small, hists[small])
        hists[large] = ctx.new_hist()
        ctx.subtract_histograms(parent, hists[small], hists[large])
        for l in (pick, right):
            best[l] = ctx.find_best_split(hists[l], *tot[l])
    _, v = ctx.refit_leaves(g, h, n_leaves=tree["num_leaves"])
    assert (v == tree["leaf_value"]).all()
