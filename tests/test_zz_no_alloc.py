"""The allocation-free histogram call (for callers that must not call cudaMalloc) against the
context-based one: same packed words, on two calls in a row that share the library's fixed
scratch array.  Collected last on purpose: a fault here cannot hide the other tests."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_09682_b200 import binding, synth

pytestmark = pytest.mark.gpu


def test_noalloc_histogram_matches_context_histogram_twice():
    n, f, nb, bits = 60_001, 28, 255, 3
    bins = synth.sweep_bins(n, f, nb, device="cuda", seed=31)
    g, h = synth.sweep_gradients(n, device="cuda", seed=32)
    ctx = binding.Context(binding.make_params(bits=bits, seed=4))
    ctx.load_binned(bins, nb)
    gq = torch.empty(n, dtype=torch.int8, device="cuda")
    hq = torch.empty(n, dtype=torch.uint8, device="cuda")
    ctx.quantize_gradients(g, h, tree=2, gq=gq, hq=hq)
    want, got = ctx.new_hist(), ctx.new_hist()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rows = synth.subset_rows(n, device="cuda", seed=33)
    before = torch.cuda.memory_allocated()
    # call 1: all rows; call 2: a row list (smaller sums: stale scratch from call 1 would show)
    ctx.build_histograms(0, want)
    binding.build_histograms_noalloc(bins, nb, gq, hq, got, status=status)
    assert torch.equal(got, want)
    ctx.build_histograms_rows(rows, want)
    binding.build_histograms_noalloc(bins, nb, gq, hq, got, rows=rows, status=status)
    assert torch.equal(got, want)
    assert int(status.item()) == 0
    assert torch.cuda.memory_allocated() == before
    # and against Algorithm 1 on the CPU
    og, oh = oracle.histogram(bins.cpu().numpy(), nb, gq.cpu().numpy(), hq.cpu().numpy(),
                              rows.cpu().numpy().astype(np.uint32))
    G, H = binding.unpack_hist(got)
    assert (G == og).all() and (H == oh).all()


def test_noalloc_strided_matrix_and_bad_entries():
    # the matrix as a view into a wider buffer (ld > n_features); then a list with one row index
    # beyond the matrix and a row with a bin code beyond n_bins: both are skipped and reported
    n, f, nb = 20_003, 12, 32
    wide = synth.sweep_bins(n, 20, nb, device="cuda", seed=41)
    bins = wide[:, 3:3 + f]                       # stride(0) = 20, stride(1) = 1
    assert bins.stride(0) == 20 and not bins.is_contiguous()
    g, h = synth.sweep_gradients(n, device="cuda", seed=42)
    q = oracle.quantize(g.cpu().numpy(), h.cpu().numpy(), bits=4, seed=6, tree=0)
    gq, hq = torch.from_numpy(q.gq).cuda(), torch.from_numpy(q.hq).cuda()
    data = bins.contiguous().cpu().numpy()
    got = torch.empty((f, nb), dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.build_histograms_noalloc(bins, nb, gq, hq, got, status=status)
    G, H = binding.unpack_hist(got)
    og, oh = oracle.histogram(data, nb, q.gq, q.hq)
    assert (G == og).all() and (H == oh).all() and int(status.item()) == 0
    rows = synth.subset_rows(n, device="cpu", seed=43).numpy().astype(np.uint32)
    bad = rows.copy()
    bad[len(bad) // 2] = n + 5                    # not a row of the matrix
    binding.build_histograms_noalloc(bins, nb, gq, hq, got, rows=torch.from_numpy(bad.view(np.int32)).cuda(), status=status)
    G, H = binding.unpack_hist(got)
    og, oh = oracle.histogram(data, nb, q.gq, q.hq, np.delete(rows, len(rows) // 2))
    assert (G == og).all() and (H == oh).all() and int(status.item()) == 1
    status.zero_()
    wide[rows[7], 3 + 2] = nb                     # one code out of range in feature 2 of row rows[7]
    binding.build_histograms_noalloc(bins, nb, gq, hq, got, rows=torch.from_numpy(rows.view(np.int32)).cuda(), status=status)
    G, H = binding.unpack_hist(got)
    og, oh = oracle.histogram(data, nb, q.gq, q.hq, rows)
    og[2, data[rows[7], 2]] -= q.gq[rows[7]]      # that one entry is missing from feature 2
    oh[2, data[rows[7], 2]] -= q.hq[rows[7]]
    assert (G == og).all() and (H == oh).all() and int(status.item()) == 1
    with pytest.raises(binding.QgbdtError) as e:  # more entries than the hessian field can take at 255 per row
        binding.build_histograms_noalloc(bins, nb, gq, hq, got, rows=torch.zeros(16_843_010, dtype=torch.int32, device="cuda"))
    assert e.value.code == binding.ERR_OVERFLOW


def test_noalloc_refuses_what_does_not_fit_its_scratch():
    bins = torch.zeros((10, 100), dtype=torch.uint8, device="cuda")
    gq = torch.zeros(10, dtype=torch.int8, device="cuda")
    hq = torch.zeros(10, dtype=torch.uint8, device="cuda")
    hist = torch.zeros((100, 255), dtype=torch.int64, device="cuda")
    with pytest.raises(binding.QgbdtError) as e:
        binding.build_histograms_noalloc(bins, 255, gq, hq, hist)       # 25500 bins > 16384
    assert e.value.code == binding.ERR_ARG and "16384" in str(e.value)
