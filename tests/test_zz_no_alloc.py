"""The allocation-free histogram call (for callers that must not call cudaMalloc) against the
context-based one: same packed words, on two calls in a row that share the library's fixed
scratch array.  Collected last on purpose: a fault here cannot hide the other tests."""
import numpy as np
import pytest
import torch

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


def test_noalloc_refuses_what_does_not_fit_its_scratch():
    bins = torch.zeros((10, 100), dtype=torch.uint8, device="cuda")
    gq = torch.zeros(10, dtype=torch.int8, device="cuda")
    hq = torch.zeros(10, dtype=torch.uint8, device="cuda")
    hist = torch.zeros((100, 255), dtype=torch.int64, device="cuda")
    with pytest.raises(binding.QgbdtError) as e:
        binding.build_histograms_noalloc(bins, 255, gq, hq, hist)       # 25500 bins > 16384
    assert e.value.code == binding.ERR_ARG and "16384" in str(e.value)
