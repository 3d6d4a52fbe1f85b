"""Pins for the CPU oracle: the paper's worked values, closed forms, invariants,
library routines and brute force.  None of these touches the CUDA path."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def rng(seed):
    return np.random.default_rng(seed)


def logistic_grads(n, seed):
    r = rng(seed)
    s = r.normal(size=n)
    y = (r.random(n) < 0.5).astype(np.float64)
    p = 1.0 / (1.0 + np.exp(-s))
    return (p - y).astype(np.float32), (p * (1 - p)).astype(np.float32)


# ----------------------------------------------------------------- Eq. 5: levels and scales

def test_levels_match_paper_counts():
    g = golden()
    for bits, key in ((2, "n_values_2bit"), (3, "n_values_3bit")):
        kg, kh = oracle.levels(bits)
        assert 2 * kg + 1 == g[key]          # signed gradient values
        assert kh + 1 == g[key]              # hessian values 0..2^B-2
        assert kh == 2 ** bits - 2           # 2^B - 2 intervals
    assert oracle.levels(3, 1) == (3, 7)     # alternative 2^B - 1 hessian levels


def test_worked_example_delta_h():
    g = golden()
    # binary classification, 3 bits: the largest hessian 0.25 must map to level 6 = 0.25 / (1/24)
    h = np.array([g["max_hessian_binary"], 0.0, 0.125], np.float32)
    q = oracle.quantize(np.zeros(3, np.float32), h, bits=3)
    assert q.hmax == 0.25
    delta_h = q.hmax / oracle.levels(3)[1]
    assert delta_h == pytest.approx(g["delta_h_3bit_binary"], rel=1e-12)
    assert q.hq.tolist() == [6, 0, 3]        # 0.125 / (1/24) = 3 exactly: integers never move
    need = 8 * delta_h ** 2 * math.log(8 / 0.01) / 0.01 ** 2
    assert round(need) == g["min_leaf_rows_example"]


def test_two_bit_value_sets():
    g, h = logistic_grads(20000, 1)
    q = oracle.quantize(g, h, bits=2, seed=3)
    assert set(np.unique(q.gq)) == {-1, 0, 1}
    assert set(np.unique(q.hq)) == {0, 1, 2}


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("mode", [0, 1])
def test_ranges_and_extreme_row(bits, mode):
    g, h = logistic_grads(5000, bits)
    q = oracle.quantize(g, h, bits=bits, seed=11, hess_levels_mode=mode)
    kg, kh = oracle.levels(bits, mode)
    assert q.gmax == np.abs(g).max() and q.hmax == h.max()
    assert q.gq.min() >= -kg and q.gq.max() <= kg
    assert q.hq.min() >= 0 and q.hq.max() <= kh
    assert abs(int(q.gq[np.abs(g).argmax()])) == kg     # the arg-max row sits on the last level
    assert int(q.hq[h.argmax()]) == kh


def test_constant_hessian_is_not_quantized():
    g = rng(0).normal(size=1000).astype(np.float32)
    q = oracle.quantize(g, None, bits=4)
    assert (q.hq == 1).all() and q.hmax == 1.0


def test_bad_values_rejected():
    g = np.array([0.1, np.nan], np.float32)
    with pytest.raises(ValueError):
        oracle.quantize(g, None, bits=3)
    with pytest.raises(ValueError):
        oracle.quantize(np.array([0.1, 0.2], np.float32), np.array([0.1, -0.2], np.float32), bits=3)
    with pytest.raises(ValueError):
        oracle.quantize(np.array([0.1, np.inf], np.float32), None, bits=3)


def test_all_zero_gradients():
    q = oracle.quantize(np.zeros(10, np.float32), np.zeros(10, np.float32), bits=3)
    assert (q.gq == 0).all() and (q.hq == 0).all()


# ----------------------------------------------------------------- Eq. 8: SR and RN

def scaled(g, gmax, k):
    """x = g / delta in float32 exactly as Eq. 6 is evaluated (one divide, one multiply)."""
    inv = np.float32(k) / np.float32(gmax)
    return np.clip((g.astype(np.float32) * inv).astype(np.float32), -k, k)


@pytest.mark.parametrize("bits", [2, 3, 5])
def test_sr_between_floor_and_ceil_and_error_bound(bits):
    g, h = logistic_grads(20000, 5)
    q = oracle.quantize(g, h, bits=bits, seed=2, tree=7)
    kg, kh = oracle.levels(bits)
    x = scaled(g, q.gmax, kg)
    assert (q.gq >= np.floor(x)).all() and (q.gq <= np.ceil(x)).all()
    y = np.clip(scaled(h, q.hmax, kh), 0, kh)
    assert (q.hq >= np.floor(y)).all() and (q.hq <= np.ceil(y)).all()
    dg = q.gmax / kg
    assert (np.abs(dg * q.gq.astype(np.float64) - g) <= dg * (1 + 1e-6)).all()   # |eps_i| <= delta_g


def test_sr_integers_never_move():
    kg = 3
    g = np.array([-3, -2, -1, 0, 1, 2, 3], np.float32)    # gmax = 3 -> delta_g = 1
    for tree in range(50):
        q = oracle.quantize(g, None, bits=3, seed=9, tree=tree)
        assert q.gq.tolist() == [-3, -2, -1, 0, 1, 2, 3]


def test_sr_is_unbiased():
    # E[g~] = g / delta_g: average over many independent (seed, tree) streams
    n, reps, bits = 400, 600, 3
    g, h = logistic_grads(n, 21)
    kg, kh = oracle.levels(bits)
    acc_g = np.zeros(n)
    acc_h = np.zeros(n)
    for r in range(reps):
        q = oracle.quantize(g, h, bits=bits, seed=100 + r // 20, tree=r % 20)
        acc_g += q.gq
        acc_h += q.hq
    xg = scaled(g, q.gmax, kg).astype(np.float64)
    xh = scaled(h, q.hmax, kh).astype(np.float64)
    for acc, x in ((acc_g, xg), (acc_h, xh)):
        mean = acc / reps
        frac = x - np.floor(x)
        sigma = np.sqrt(frac * (1 - frac) / reps) + 1e-9
        z = (mean - x) / sigma
        assert np.abs(z).max() < 5.0
        assert abs(z.mean()) < 0.3            # no systematic drift up or down
    # E[G~ delta_g] = G and E[H~ delta_h] = H
    assert abs(acc_g.sum() / reps * q.gmax / kg - g.sum(dtype=np.float64)) < 4 * q.gmax / kg * math.sqrt(n / reps)


def test_sr_sum_error_within_hoeffding_bound():
    # proof of Theorem 5.3: |sum eps_i| <= delta_g sqrt(2 n ln(4/delta)) with prob >= 1 - delta/2
    n, delta, bits = 20000, 0.1, 3
    g, _ = logistic_grads(n, 33)
    kg, _ = oracle.levels(bits)
    fails = 0
    trials = 60
    for t in range(trials):
        q = oracle.quantize(g, None, bits=bits, seed=77, tree=t)
        dg = q.gmax / kg
        err = abs(dg * q.gq.astype(np.float64).sum() - g.astype(np.float64).sum())
        fails += err > dg * math.sqrt(2 * n * math.log(4 / delta))
    assert fails <= trials * delta / 2 + 3


def test_rn_matches_floor_plus_half():
    g, h = logistic_grads(5000, 8)
    q = oracle.quantize(g, h, bits=4, rounding=1)
    kg, kh = oracle.levels(4)
    x = scaled(g, q.gmax, kg)
    f = np.floor(x)
    assert (q.gq == f + ((x - f) >= 0.5)).all()
    # ties go up (Eq. 8): x = -0.5 -> 0, x = 0.5 -> 1, x = 2.5 -> 3  (gmax = 7 -> delta = 1)
    q = oracle.quantize(np.array([7, -0.5, 0.5, 2.5, -2.5], np.float32), None, bits=4, rounding=1)
    assert q.gq.tolist() == [7, 0, 1, 3, -2]


def test_rn_is_biased_where_sr_is_not():
    # the paper's motivation for SR: with values clustered below half a level RN loses the whole sum
    g = np.full(4000, 0.1, np.float32)
    g[0] = 1.0                                  # gmax = 1, delta_g = 1 at 2 bits
    rn = oracle.quantize(g, None, bits=2, rounding=1).gq.astype(np.int64).sum()
    sr = oracle.quantize(g, None, bits=2, rounding=0, seed=5).gq.astype(np.int64).sum()
    assert rn == 1
    assert abs(sr - g.astype(np.float64).sum()) < 5 * math.sqrt(4000 * 0.09)


# ----------------------------------------------------------------- the counter hash (statistical pins)

def test_hash_uniform_and_independent():
    n = 1 << 18
    ug, uh = oracle.sr_uniforms(20220709, 3, 0, n)
    assert ug.max() < (1 << 24) and uh.max() < (1 << 24)
    for u in (ug, uh):
        counts = np.bincount(u >> 16, minlength=256)            # top byte
        chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 255 + 6 * math.sqrt(2 * 255)
        counts = np.bincount(u & 0xFF, minlength=256)           # low byte
        chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 255 + 6 * math.sqrt(2 * 255)
        x = u.astype(np.float64) / (1 << 24)
        assert abs(x.mean() - 0.5) < 5 / math.sqrt(12 * n)
        assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 5 / math.sqrt(n)     # lag-1 over rows
    a = ug.astype(np.float64)
    b = uh.astype(np.float64)
    assert abs(np.corrcoef(a, b)[0, 1]) < 5 / math.sqrt(n)                  # u_g vs u_h
    joint = np.bincount((ug >> 20) * 16 + (uh >> 20), minlength=256)
    chi2 = ((joint - n / 256) ** 2 / (n / 256)).sum()
    assert chi2 < 255 + 6 * math.sqrt(2 * 255)


def test_hash_streams_differ_by_tree_seed_and_row_offset():
    a, _ = oracle.sr_uniforms(1, 0, 0, 4096)
    b, _ = oracle.sr_uniforms(1, 1, 0, 4096)
    c, _ = oracle.sr_uniforms(2, 0, 0, 4096)
    d, _ = oracle.sr_uniforms(1 + (1 << 32), 0, 0, 4096)
    for other in (b, c, d):
        assert (a == other).mean() < 0.01
        assert abs(np.corrcoef(a.astype(float), other.astype(float))[0, 1]) < 0.08
    e, _ = oracle.sr_uniforms(1, 0, 100, 64)          # keyed by absolute row id
    assert (e == a[100:164]).all()


# ----------------------------------------------------------------- Algorithm 1

def small_problem(n=700, J=5, nb=11, bits=3, seed=0):
    r = rng(seed)
    data = r.integers(0, nb, size=(n, J), dtype=np.uint8)
    g, h = logistic_grads(n, seed + 1)
    q = oracle.quantize(g, h, bits=bits, seed=seed)
    return data, q, g, h


def test_histogram_brute_force_and_bincount():
    data, q, _, _ = small_problem()
    n, J = data.shape
    nb = 11
    idx = np.sort(rng(4).choice(n, size=300, replace=False)).astype(np.uint32)
    for rows in (None, idx):
        hg, hh = oracle.histogram(data, nb, q.gq, q.hq, rows)
        sel = np.arange(n) if rows is None else rows
        for j in range(J):
            for b in range(nb):
                m = data[sel, j] == b
                assert hg[j, b] == q.gq[sel][m].astype(np.int64).sum()
                assert hh[j, b] == q.hq[sel][m].astype(np.int64).sum()
            assert (np.bincount(data[sel, j], weights=q.gq[sel], minlength=nb) == hg[j]).all()
            assert (np.bincount(data[sel, j], weights=q.hq[sel], minlength=nb) == hh[j]).all()


def test_histogram_invariants():
    data, q, _, _ = small_problem(n=2000, J=7, nb=16)
    n = data.shape[0]
    perm = rng(9).permutation(n).astype(np.uint32)
    hg, hh = oracle.histogram(data, 16, q.gq, q.hq)
    hg2, hh2 = oracle.histogram(data, 16, q.gq, q.hq, perm)            # row order does not matter
    assert (hg == hg2).all() and (hh == hh2).all()
    assert (hg.sum(axis=1) == q.gq.astype(np.int64).sum()).all()        # every feature sums to the leaf total
    assert (hh.sum(axis=1) == q.hq.astype(np.int64).sum()).all()
    left, right = perm[:777], perm[777:]
    lg, lh = oracle.histogram(data, 16, q.gq, q.hq, left)
    rg, rh = oracle.histogram(data, 16, q.gq, q.hq, right)
    assert (lg + rg == hg).all() and (lh + rh == hh).all()              # parent = left + right
    ones = np.ones(n, np.uint8)
    _, cnt = oracle.histogram(data, 16, q.gq, ones)
    for j in range(7):
        assert (cnt[j] == np.bincount(data[:, j], minlength=16)).all()  # constant hessian: plain counts
    eg, eh = oracle.histogram(data, 16, q.gq, q.hq, np.zeros(0, np.uint32))
    assert not eg.any() and not eh.any()                                # empty leaf


def test_histogram_rejects_out_of_range_bin():
    data, q, _, _ = small_problem()
    with pytest.raises(ValueError):
        oracle.histogram(data, 10, q.gq, q.hq)


# ----------------------------------------------------------------- partition

def test_partition_is_stable_filter():
    data, _, _, _ = small_problem(n=3000, J=6, nb=13)
    idx = rng(2).permutation(3000)[:1700].astype(np.uint32)
    for f, t in ((0, 5), (3, 0), (5, 12), (2, 11)):
        out, nl = oracle.partition(data, idx, f, t)
        key = data[idx, f] > t
        ref = idx[np.argsort(key, kind="stable")]
        assert (out == ref).all()
        assert nl == int((~key).sum())
        assert sorted(out.tolist()) == sorted(idx.tolist())


# ----------------------------------------------------------------- Eq. 7 and the scan

def exact_gain(gl, hl, gr, hr, dg, dh):
    """Eq. 7 in exact rational arithmetic."""
    def term(G, H):
        return (Fraction(G) * dg) ** 2 / (2 * Fraction(H) * dh)
    return term(gl, hl) + term(gr, hr) - term(gl + gr, hl + hr)


def test_gain_matches_exact_rational_eq7():
    r = rng(12)
    dg, dh = Fraction(1, 3), Fraction(1, 24)
    for _ in range(200):
        gl, gr = (int(v) for v in r.integers(-5000, 5000, 2))
        hl, hr = (int(v) for v in r.integers(1, 9000, 2))
        got = oracle.gain(gl, hl, gr, hr, float(dg), float(dh))
        want = float(exact_gain(gl, hl, gr, hr, dg, dh))
        assert got == pytest.approx(want, rel=1e-9, abs=1e-9)
    # closed forms: equal and opposite children; identical children give zero gain
    assert oracle.gain(10, 5, -10, 5, 1.0, 1.0) == pytest.approx(20.0)
    assert oracle.gain(7, 3, 7, 3, 0.5, 0.25) == pytest.approx(0.0, abs=1e-12)
    # lambda enters only the denominators
    assert oracle.gain(10, 5, -10, 5, 1.0, 1.0, 5.0) == pytest.approx(0.5 * (10 + 10 - 0))


def brute_force_split(data, nb, gq, hq, sel, dg, dh, min_data, const_h):
    """Best (gain, feature, bin) straight from the rows, never forming a histogram."""
    G, H, n_s = int(gq[sel].sum()), int(hq[sel].sum()), len(sel)
    best = None
    for f in range(data.shape[1]):
        for t in range(nb - 1):
            m = data[sel, f] <= t
            gl, hl = int(gq[sel][m].sum()), int(hq[sel][m].sum())
            gr, hr = G - gl, H - hl
            if hl <= 0 or hr <= 0:
                continue
            nl = hl if const_h else (hl * n_s + H // 2) // H
            if nl < min_data or n_s - nl < min_data:
                continue
            gain = float(exact_gain(gl, hl, gr, hr, Fraction(dg), Fraction(dh)))
            if gain <= 0:
                continue
            if best is None or gain > best[0] * (1 + 1e-12):
                best = (gain, f, t, gl, hl, nl)
    return best


@pytest.mark.parametrize("const_h", [False, True])
def test_find_split_brute_force_from_rows(const_h):
    data, q, g, h = small_problem(n=900, J=4, nb=9, bits=3, seed=3)
    if const_h:
        q = oracle.quantize(g, None, bits=3, seed=3)
    gq, hq = q.gq.astype(np.int64), q.hq.astype(np.int64)
    sel = np.arange(900)[::2]
    hg, hh = oracle.histogram(data, 9, q.gq, q.hq, sel.astype(np.uint32))
    prm = oracle.make_params(bits=3, min_data_in_leaf=20)
    s = oracle.find_split(hg, hh, gq[sel].sum(), hq[sel].sum(), len(sel), q.gmax, q.hmax, const_h, prm)
    kg, kh = oracle.levels(3)
    dg = q.gmax / kg
    dh = 1.0 if const_h else q.hmax / kh
    ref = brute_force_split(data, 9, gq, hq, sel, dg, dh, 20, const_h)
    assert s.valid and ref is not None
    assert (s.feature, s.bin) == (ref[1], ref[2])
    assert s.gain == pytest.approx(ref[0], rel=1e-9)
    assert (s.gl, s.hl, s.nl_est) == (ref[3], ref[4], ref[5])
    assert s.gl + s.gr == gq[sel].sum() and s.hl + s.hr == hq[sel].sum()
    assert s.nl_est + s.nr_est == len(sel)
    if const_h:
        assert s.nl_est == int((data[sel, s.feature] <= s.bin).sum())       # counts are exact


def test_find_split_ties_take_lowest_feature_then_bin():
    nb = 6
    hg = np.zeros((3, nb), np.int64)
    hh = np.zeros((3, nb), np.int64)
    hg[:, 1], hg[:, 4] = 30, -30                 # every feature identical: thresholds 1,2,3 tie
    hh[:, 1], hh[:, 4] = 40, 40
    prm = oracle.make_params(bits=3, min_data_in_leaf=1)
    s = oracle.find_split(hg, hh, 0, 80, 80, 1.0, 1.0, False, prm)
    assert (s.feature, s.bin) == (0, 1)
    hg[0] = 0
    hh[0] = 0
    hh[0, 0] = 80                                 # feature 0 now has nothing on the right: invalid
    s = oracle.find_split(hg, hh, 0, 80, 80, 1.0, 1.0, False, prm)
    assert (s.feature, s.bin) == (1, 1)


def test_find_split_validity_rules():
    nb = 4
    hg = np.array([[5, -5, 0, 0]], np.int64)
    hh = np.array([[10, 10, 0, 0]], np.int64)
    ok = oracle.find_split(hg, hh, 0, 20, 20, 1.0, 1.0, True, oracle.make_params(min_data_in_leaf=10))
    assert ok.valid and (ok.feature, ok.bin) == (0, 0)
    no = oracle.find_split(hg, hh, 0, 20, 20, 1.0, 1.0, True, oracle.make_params(min_data_in_leaf=11))
    assert not no.valid                           # too few rows on a side
    no = oracle.find_split(hg, hh, 0, 20, 20, 1.0, 1.0, True,
                           oracle.make_params(min_data_in_leaf=1, min_sum_hessian=10.5))
    assert not no.valid                           # hessian mass too small
    no = oracle.find_split(hg, hh, 0, 20, 20, 1.0, 1.0, True,
                           oracle.make_params(min_data_in_leaf=1, min_gain=1e9))
    assert not no.valid                           # gain must exceed the floor
    # a side whose hessian mass is zero is never a candidate (Eq. 7 would divide by zero)
    z = oracle.find_split(np.array([[5, -5, 0, 0]], np.int64), np.array([[0, 20, 0, 0]], np.int64), 0, 20, 20,
                          1.0, 1.0, False, oracle.make_params(min_data_in_leaf=0))
    assert not z.valid
    # estimated rows per side are rounded to nearest: 7/20 of 30 rows = 10.5 -> 11
    hg2 = np.array([[9, -9, 0, 0]], np.int64)
    hh2 = np.array([[7, 13, 0, 0]], np.int64)
    e = oracle.find_split(hg2, hh2, 0, 20, 30, 1.0, 1.0, False, oracle.make_params(min_data_in_leaf=11))
    assert e.valid and (e.nl_est, e.nr_est) == (11, 19)
    flat = oracle.find_split(np.zeros((1, nb), np.int64), hh, 0, 20, 20, 1.0, 1.0, True,
                             oracle.make_params(min_data_in_leaf=1))
    assert not flat.valid                         # zero gain is not a split


def test_high_bitwidth_agrees_with_full_precision_split():
    # well separated data: feature 2 carries a step in the gradient; 8-bit SR must find the same
    # (feature, bin) as the unquantized float64 criterion (Eq. 4)
    r = rng(40)
    n, J, nb = 6000, 5, 32
    data = r.integers(0, nb, size=(n, J), dtype=np.uint8)
    g = (np.where(data[:, 2] <= 13, -0.6, 0.5) + 0.05 * r.normal(size=n)).astype(np.float32)
    h = np.full(n, 0.2, np.float32) + 0.01 * r.random(n).astype(np.float32)
    best = None
    G, H = g.astype(np.float64).sum(), h.astype(np.float64).sum()
    for f in range(J):
        for t in range(nb - 1):
            m = data[:, f] <= t
            gl, hl = g[m].astype(np.float64).sum(), h[m].astype(np.float64).sum()
            gain = gl * gl / (2 * hl) + (G - gl) ** 2 / (2 * (H - hl)) - G * G / (2 * H)
            if best is None or gain > best[0]:
                best = (gain, f, t)
    q = oracle.quantize(g, h, bits=8, seed=4)
    hg, hh = oracle.histogram(data, nb, q.gq, q.hq)
    s = oracle.find_split(hg, hh, q.gq.astype(np.int64).sum(), q.hq.astype(np.int64).sum(), n, q.gmax, q.hmax,
                          False, oracle.make_params(bits=8))
    assert (s.feature, s.bin) == (best[1], best[2]) == (2, 13)
    assert s.gain == pytest.approx(best[0], rel=0.02)      # dequantized gain approximates the FP gain


# ----------------------------------------------------------------- Eq. 9 (theory): the printed numbers

def eq9_bound(bits, n_s, n1, n2, gmax, eps, gamma, delta):
    a = gmax * math.sqrt(2 * math.log(4 / delta)) / (gamma ** 2 * eps * 2 ** (bits - 1))
    a *= math.sqrt(1 / n1) + math.sqrt(1 / n2)
    b = gmax ** 2 * math.log(4 / delta) / (gamma ** 2 * eps ** 2 * n_s * 4 ** (bits - 2))
    return a + b


def test_eq9_printed_values():
    g = golden()
    b3 = eq9_bound(3, 1e7, 5e6, 5e6, 1.0, 0.1, 0.2, 0.1)
    b4 = eq9_bound(4, 1e7, 5e6, 5e6, 1.0, 0.1, 0.2, 0.1)
    assert b3 == pytest.approx(g["eq9_bound_3bit"], abs=0.005)
    assert b4 < g["eq9_bound_4bit_below"] and b4 > 0.07


def test_quantized_gain_error_within_eq9_bound():
    # constant hessian, a leaf with a clear split: the relative change of G(s -> s1, s2) caused by
    # SR stays under Eq. 9's bound in at least 1 - delta of the trials
    r = rng(50)
    n, bits, delta = 40000, 3, 0.1
    side = r.random(n) < 0.5
    g = (np.where(side, 0.4, -0.4) + 0.2 * r.normal(size=n)).astype(np.float32)
    g64 = g.astype(np.float64)
    n1, n2 = int(side.sum()), int((~side).sum())
    G_true = g64[side].sum() ** 2 / (2 * n1) + g64[~side].sum() ** 2 / (2 * n2)
    gamma = (abs(g64[side].sum()) + abs(g64[~side].sum())) / (2 * np.abs(g64).sum())
    kg, _ = oracle.levels(bits)
    fails, trials = 0, 40
    for t in range(trials):
        q = oracle.quantize(g, None, bits=bits, seed=91, tree=t)
        dg = q.gmax / kg
        gq = q.gq.astype(np.float64)
        G_q = (dg * gq[side].sum()) ** 2 / (2 * n1) + (dg * gq[~side].sum()) ** 2 / (2 * n2)
        eps = np.abs(g64).mean() * 0.999
        bound = eq9_bound(bits, n, n1, n2, q.gmax, eps, gamma, delta)
        fails += abs(G_q - G_true) / G_true > bound
    assert fails <= trials * delta + 2


# ----------------------------------------------------------------- Eq. 3: refit

def test_refit_closed_form():
    g, h = logistic_grads(5000, 60)
    idx = np.arange(5000, dtype=np.uint32)
    w, v = oracle.refit(g, h, idx)
    want = -math.fsum(g.astype(np.float64)) / math.fsum(h.astype(np.float64))
    assert w == pytest.approx(want, rel=1e-7)
    assert w == pytest.approx(-g.astype(np.float64).mean() / h.astype(np.float64).mean(), rel=1e-7)
    sub = idx[100:900]
    w, v = oracle.refit(g, h, sub, lambda_l2=2.0, learning_rate=0.1)
    want = -math.fsum(g[sub].astype(np.float64)) / (math.fsum(h[sub].astype(np.float64)) + 2.0)
    assert w == pytest.approx(want, rel=1e-7)
    assert v == np.float32(0.1 * w)
    w, _ = oracle.refit(g, None, sub)              # constant hessian 1: minus the mean gradient
    assert w == pytest.approx(-g[sub].astype(np.float64).mean(), rel=1e-7)
    w1, _ = oracle.refit(g, h, sub[::-1].copy())   # order-independent, bit for bit
    w2, _ = oracle.refit(g, h, sub)
    assert w1 == w2
    assert oracle.refit(g, np.zeros_like(h), sub)[0] == 0.0   # empty hessian mass: defined as 0


# ----------------------------------------------------------------- Eq. 1: gradients

def test_sigmoid_accuracy_symmetry_monotone():
    xs = np.concatenate([np.linspace(-45, 45, 4001), rng(1).normal(size=2000) * 3]).astype(np.float32)
    got = np.array([oracle.sigmoid(float(x)) for x in xs], np.float64)
    want = 1.0 / (1.0 + np.exp(-xs.astype(np.float64)))
    assert np.abs(got - want).max() < 2e-7
    rel = np.abs(got - want) / want
    assert rel[xs > -40].max() < 1e-6
    assert oracle.sigmoid(0.0) == 0.5
    order = np.argsort(xs, kind="stable")
    assert (np.diff(got[order]) >= -1.2e-7).all()
    for x in (0.3, 1.7, 9.0, 33.0):
        assert oracle.sigmoid(x) + oracle.sigmoid(-x) == pytest.approx(1.0, abs=1.2e-7)


def test_gradients_definitions_and_ranges():
    r = rng(70)
    s = (r.normal(size=3000) * 4).astype(np.float32)
    y = (r.random(3000) < 0.5).astype(np.float32)
    g, h = oracle.gradients(0, s, y)
    p = 1 / (1 + np.exp(-s.astype(np.float64)))
    assert np.abs(g - (p - y)).max() < 3e-7
    assert np.abs(h - p * (1 - p)).max() < 3e-7
    assert np.abs(g).max() <= 1.0 and h.max() <= 0.25 and h.min() >= 0.0     # the paper's ranges
    g2, h2 = oracle.gradients(1, s, y)
    assert h2 is None and (g2 == s - y).all()


# ----------------------------------------------------------------- training loop

def toy_classification(n=4000, J=6, nb=32, seed=0):
    r = rng(seed)
    x = r.normal(size=(n, J))
    edges = np.quantile(x, np.linspace(0, 1, nb + 1)[1:-1], axis=0)
    data = np.stack([np.searchsorted(edges[:, j], x[:, j]) for j in range(J)], axis=1).astype(np.uint8)
    y = ((x[:, 0] + 0.7 * x[:, 1] * x[:, 2] + 0.3 * r.normal(size=n)) > 0).astype(np.float32)
    return data, y, x


def logloss(s, y):
    p = 1 / (1 + np.exp(-s.astype(np.float64)))
    return float(-(y * np.log(p + 1e-12) + (1 - y) * np.log(1 - p + 1e-12)).mean())


def test_tree_structure_is_consistent():
    data, y, _ = toy_classification()
    prm = oracle.make_params(bits=3, num_leaves=15, min_data_in_leaf=20, seed=5)
    scores = np.zeros(len(y), np.float32)
    t, row_leaf = oracle.train_tree(data, 32, y, scores, prm, 0, want_row_leaf=True)
    assert 2 <= t.num_leaves <= 15
    assert t.leaf_count.sum() == len(y) and (t.leaf_count >= 1).all()
    assert (np.bincount(row_leaf, minlength=t.num_leaves) == t.leaf_count).all()
    assert (oracle.predict_leaf(data, t) == row_leaf).all()          # node wiring routes rows to their leaf
    assert (scores == t.leaf_value[row_leaf]).all()                  # score update = leaf output
    # best-first: when node i was made, every leaf that already existed had a gain no larger than
    # node i's; a later node j split such a leaf iff its parent node was made before i (gains are
    # not monotone over the whole sequence: a child's gain may exceed its parent's)
    parent = np.full(t.num_leaves - 1, -1)
    for i in range(t.num_leaves - 1):
        for c in (t.left[i], t.right[i]):
            if c >= 0:
                parent[c] = i
    for i in range(t.num_leaves - 1):
        for j in range(i + 1, t.num_leaves - 1):
            if parent[j] < i:
                assert t.gain[j] <= t.gain[i]
    # every internal node's children are either nodes created later or leaves
    for i in range(t.num_leaves - 1):
        for c in (t.left[i], t.right[i]):
            assert c < 0 or c > i
    # leaf values are Eq. 3 on the original gradients
    g, h = oracle.gradients(0, np.zeros(len(y), np.float32), y)
    for l in range(t.num_leaves):
        rows = np.nonzero(row_leaf == l)[0]
        w = -g[rows].astype(np.float64).sum() / h[rows].astype(np.float64).sum()
        assert t.leaf_value[l] == pytest.approx(0.1 * w, rel=1e-6)


def test_first_split_is_the_root_argmax():
    data, y, _ = toy_classification(seed=3)
    prm = oracle.make_params(bits=4, num_leaves=2, seed=8)
    scores = np.zeros(len(y), np.float32)
    t = oracle.train_tree(data, 32, y, scores, prm, 0)
    g, h = oracle.gradients(0, np.zeros(len(y), np.float32), y)
    q = oracle.quantize(g, h, bits=4, seed=8, tree=0)
    hg, hh = oracle.histogram(data, 32, q.gq, q.hq)
    s = oracle.find_split(hg, hh, q.gq.astype(np.int64).sum(), q.hq.astype(np.int64).sum(), len(y), q.gmax, q.hmax,
                          False, prm)
    assert (t.feature[0], t.bin[0]) == (s.feature, s.bin) and t.gain[0] == s.gain
    assert t.leaf_count[0] == int((data[:, s.feature] <= s.bin).sum())


def test_every_split_is_the_best_first_choice():
    # replay the growth from the recorded nodes: at each step the split taken must be the largest-gain
    # candidate among the current leaves, each found from that leaf's own rows and integer totals
    data, y, _ = toy_classification(n=3000, seed=6)
    prm = oracle.make_params(bits=3, num_leaves=6, seed=4)
    scores = np.zeros(len(y), np.float32)
    t = oracle.train_tree(data, 32, y, scores, prm, 0)
    g, h = oracle.gradients(0, np.zeros(len(y), np.float32), y)
    q = oracle.quantize(g, h, bits=3, seed=4, tree=0)
    gq, hq = q.gq.astype(np.int64), q.hq.astype(np.int64)

    def best_of(rows):
        hg, hh = oracle.histogram(data, 32, q.gq, q.hq, rows.astype(np.uint32))
        return oracle.find_split(hg, hh, gq[rows].sum(), hq[rows].sum(), len(rows), q.gmax, q.hmax, False, prm)

    leaves = {0: np.arange(len(y))}
    for node in range(t.num_leaves - 1):
        cands = {l: best_of(r) for l, r in leaves.items()}
        pick = max((l for l in cands if cands[l].valid), key=lambda l: (cands[l].gain, -l))
        s = cands[pick]
        assert (t.feature[node], t.bin[node]) == (s.feature, s.bin) and t.gain[node] == s.gain
        rows = leaves[pick]
        go_left = data[rows, s.feature] <= s.bin
        assert gq[rows[go_left]].sum() == s.gl and hq[rows[go_left]].sum() == s.hl
        leaves[pick], leaves[node + 1] = rows[go_left], rows[~go_left]
    for l, rows in leaves.items():
        assert t.leaf_count[l] == len(rows)


def test_training_loss_decreases_and_tracks_high_precision():
    data, y, _ = toy_classification(n=6000, seed=1)
    losses = {}
    for bits in (2, 3, 8):
        prm = oracle.make_params(bits=bits, num_leaves=15, num_trees=12, seed=3)
        scores = np.zeros(len(y), np.float32)
        seq = [logloss(scores, y)]
        for k in range(12):
            oracle.train_tree(data, 32, y, scores, prm, k)
            seq.append(logloss(scores, y))
        assert all(b < a for a, b in zip(seq, seq[1:]))               # monotone on the training set
        losses[bits] = seq[-1]
    assert losses[2] < 0.62 and abs(losses[2] - losses[8]) < 0.03     # low bits ~ high bits (Table 2's claim)
    assert abs(losses[3] - losses[8]) < 0.02


def test_regression_constant_hessian_training():
    r = rng(5)
    n = 5000
    data = r.integers(0, 16, size=(n, 4), dtype=np.uint8)
    y = (1.5 * (data[:, 1] > 7) - 0.8 * (data[:, 3] > 3) + 0.05 * r.normal(size=n)).astype(np.float32)
    prm = oracle.make_params(bits=4, objective=1, num_leaves=4, num_trees=1, learning_rate=1.0, seed=2)
    scores = np.zeros(n, np.float32)
    t = oracle.train_tree(data, 16, y, scores, prm, 0)
    assert t.num_leaves == 4
    assert {(int(f), int(b)) for f, b in zip(t.feature, t.bin)} == {(1, 7), (3, 3)}
    assert float(((scores - y) ** 2).mean()) < 0.01                   # lr 1: the four step levels are recovered


def test_train_stops_when_no_valid_split():
    data = np.zeros((100, 3), np.uint8)                               # one bin only: nothing to split
    y = (np.arange(100) % 2).astype(np.float32)
    scores = np.zeros(100, np.float32)
    t = oracle.train_tree(data, 4, y, scores, oracle.make_params(num_leaves=8), 0)
    assert t.num_leaves == 1 and t.leaf_count[0] == 100
    assert abs(float(t.leaf_value[0])) < 1e-6                         # balanced labels: w = 0


def test_multi_tree_wrapper_is_the_loop_over_single_trees():
    # qo_train is only a loop over qo_train_tree that lays the trees out one after the other
    import ctypes as C
    data, y, _ = toy_classification(seed=9)
    n, L, K = len(y), 7, 3
    prm = oracle.make_params(bits=3, num_leaves=L, num_trees=K, seed=21)
    want_scores = np.zeros(n, np.float32)
    want = oracle.train(data, 32, y, want_scores, prm)
    scores = np.zeros(n, np.float32)
    leaves = np.zeros(K, np.int32)
    nf, nb_, nl, nr = (np.zeros(K * (L - 1), np.int32) for _ in range(4))
    ng = np.zeros(K * (L - 1), np.float64)
    lv, lc = np.zeros(K * L, np.float32), np.zeros(K * L, np.int64)
    p = lambda a, t: a.ctypes.data_as(C.POINTER(t))
    d = np.ascontiguousarray(data, np.uint8)
    rc = oracle.lib().qo_train(p(d, C.c_uint8), C.c_int64(n), d.shape[1], 32, p(y, C.c_float), p(scores, C.c_float),
                               C.byref(prm), p(leaves, C.c_int32), p(nf, C.c_int32), p(nb_, C.c_int32),
                               p(nl, C.c_int32), p(nr, C.c_int32), p(ng, C.c_double), p(lv, C.c_float),
                               p(lc, C.c_int64))
    assert rc == 0
    assert (scores == want_scores).all()
    for k, t in enumerate(want):
        m = t.num_leaves
        assert leaves[k] == m
        s_ = slice(k * (L - 1), k * (L - 1) + m - 1)
        assert (nf[s_] == t.feature).all() and (nb_[s_] == t.bin).all() and (nl[s_] == t.left).all()
        assert (nr[s_] == t.right).all() and (ng[s_] == t.gain).all()
        assert (lv[k * L:k * L + m] == t.leaf_value).all() and (lc[k * L:k * L + m] == t.leaf_count).all()


def test_leaf_value_from_quantized_sums_is_the_closed_form():
    # Sec. 4.2: w~ = -(G~ delta_g) / (H~ delta_h); exact rational arithmetic as the reference
    from fractions import Fraction
    r = np.random.default_rng(4)
    for bits, mode, const_h in ((2, 0, False), (3, 0, False), (4, 1, False), (5, 0, True), (8, 0, False)):
        kg, kh = oracle.levels(bits, mode)
        for _ in range(20):
            G, H = int(r.integers(-10**6, 10**6)), int(r.integers(1, 10**7))
            gmax, hmax = np.float32(r.uniform(0.1, 3.0)), np.float32(r.uniform(0.01, 0.25))
            lam = float(r.choice([0.0, 0.5]))
            w, v = oracle.leaf_value_quantized(G, H, float(gmax), float(hmax), bits, mode, const_h, lam, 0.1)
            dg = Fraction(float(gmax)) / kg
            dh = Fraction(1) if const_h else Fraction(float(hmax)) / kh
            exact = -(G * dg) / (H * dh + Fraction(lam))
            assert w == pytest.approx(float(exact), rel=1e-14)
            assert v == np.float32(0.1 * w)
    # no admissible denominator: value 0 (an empty leaf with no regulariser)
    assert oracle.leaf_value_quantized(5, 0, 1.0, 1.0, 3)[0] == 0.0


def test_unrefitted_tree_has_the_same_structure_and_close_values():
    # the leaf-value rule does not touch the growth of the tree; at 8 bits w~ is within the
    # quantization error of the refitted value (E[G~ delta_g] = G, Sec. 4.2), at 2 bits it is coarser
    data, y, _ = toy_classification(seed=11)
    for bits, tol in ((8, 0.03), (2, 0.6)):
        prm = oracle.make_params(bits=bits, num_leaves=8, seed=13, learning_rate=1.0)
        s1, s2 = np.zeros(len(y), np.float32), np.zeros(len(y), np.float32)
        a = oracle.train_tree(data, 32, y, s1, prm, 0)
        b, row_leaf = oracle.train_tree(data, 32, y, s2, prm, 0, want_row_leaf=True, refit=False)
        assert a.num_leaves == b.num_leaves and (a.feature == b.feature).all() and (a.bin == b.bin).all()
        assert (a.leaf_count == b.leaf_count).all()
        assert np.abs(a.leaf_value - b.leaf_value).max() < tol * np.abs(a.leaf_value).max()
        assert (s2 == b.leaf_value[row_leaf]).all()
        # each value is the closed form on the leaf's own integer sums
        g, h = oracle.gradients(0, np.zeros(len(y), np.float32), y)
        q = oracle.quantize(g, h, bits=bits, seed=13, tree=0)
        for l in range(b.num_leaves):
            rows = np.nonzero(row_leaf == l)[0]
            G, H = int(q.gq[rows].astype(np.int64).sum()), int(q.hq[rows].astype(np.int64).sum())
            assert b.leaf_value[l] == oracle.leaf_value_quantized(G, H, q.gmax, q.hmax, bits, learning_rate=1.0)[1]


def test_floating_point_histogram_is_the_weighted_bincount():
    # Algorithm 1 with the original gradients: per feature a bincount weighted by g resp. h
    # (library routine), and the quantized histogram times the interval length approximates it
    r = np.random.default_rng(8)
    n, J, nb = 5000, 6, 11
    data = r.integers(0, nb, size=(n, J), dtype=np.uint8)
    g = r.normal(size=n).astype(np.float32)
    h = r.uniform(0.01, 0.25, size=n).astype(np.float32)
    idx = np.sort(r.choice(n, 1800, replace=False)).astype(np.uint32)
    for rows in (None, idx):
        hg, hh = oracle.histogram_fp(data, nb, g, h, rows)
        sel = np.arange(n) if rows is None else rows
        for j in range(J):
            assert np.allclose(hg[j], np.bincount(data[sel, j], weights=g[sel].astype(np.float64), minlength=nb), rtol=1e-12, atol=1e-12)
            assert np.allclose(hh[j], np.bincount(data[sel, j], weights=h[sel].astype(np.float64), minlength=nb), rtol=1e-12, atol=1e-12)
    hg1, hh1 = oracle.histogram_fp(data, nb, g, None)
    assert (hh1 == np.stack([np.bincount(data[:, j], minlength=nb) for j in range(J)])).all()   # constant hessian: counts
    # E[G~ delta_g] = G (Sec. 4.2): at 8 bits the dequantized integer histogram is close to the floating-point one
    q = oracle.quantize(g, h, bits=8, seed=3)
    ig, ih = oracle.histogram(data, nb, q.gq, q.hq)
    kg, kh = oracle.levels(8)
    hg, hh = oracle.histogram_fp(data, nb, g, h)
    assert np.abs(ig * (q.gmax / kg) - hg).max() < 0.02 * np.abs(hg).max() + 1.0
    assert np.abs(ih * (q.hmax / kh) - hh).max() < 0.02 * hh.max()
