"""Seeded synthetic inputs shaped like the paper's workloads (Table 1 shapes).

This module only draws random numbers and bins them; it holds none of the method's
arithmetic (no quantizer, histogram, gain, refit), so both the CUDA path and the CPU
checker may be fed from it.  Everything is generated with torch on the device asked
for and returned as torch tensors; ``rows`` lets a test shrink a configuration while
keeping its structure.

Configurations (names follow the benchmark description):
  tiny    50,000 x 28, 64 quantile bins, linear-logit labels, logistic, 2-bit, 31 leaves
  tall    1,000,000 x 28, 255 bins, labels from a random depth-6 tree + 10% flips, 3-bit
  wide    400,000 x 2,000, 255 bins, sparse linear-logit labels, 3-bit
  large   10,500,000 x 28, 255 bins, sum of 8 step functions + noise, squared loss, 4-bit
  sweep   uniform bin codes with 90% of the mass in bin 0 for the odd features,
          gradients of random logits against random labels
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

MASTER_SEED = 20220709


@dataclass
class Workload:
    name: str
    bins: torch.Tensor          # uint8 [N, F], row-major bin codes
    n_bins: int
    labels: torch.Tensor        # float32 [N]
    params: dict = field(default_factory=dict)   # keyword arguments of the training parameters


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def quantile_bin(x: torch.Tensor, n_bins: int) -> torch.Tensor:
    """Per-feature equal-frequency binning of a float matrix [N, F] into uint8 codes."""
    n, f = x.shape
    out = torch.empty((n, f), dtype=torch.uint8, device=x.device)
    cut = (torch.arange(1, n_bins, device=x.device, dtype=torch.float64) * n / n_bins).long().clamp_(0, n - 1)
    for j in range(f):
        col = x[:, j].contiguous()
        edges = torch.sort(col).values[cut]
        out[:, j] = torch.bucketize(col, edges, right=False).to(torch.uint8)
    return out


def _normal_binned(n, f, n_bins, gen, device, want_x=True, chunk=64):
    """N(0,1) features, quantile-binned; returns (x or None, codes)."""
    codes = torch.empty((n, f), dtype=torch.uint8, device=device)
    xs = [] if want_x else None
    for j0 in range(0, f, chunk):
        j1 = min(f, j0 + chunk)
        x = torch.randn((n, j1 - j0), generator=gen, device=device, dtype=torch.float32)
        codes[:, j0:j1] = quantile_bin(x, n_bins)
        if want_x:
            xs.append(x)
    return (torch.cat(xs, dim=1) if want_x else None), codes


def tiny(device="cpu", rows=50_000, seed=MASTER_SEED + 1) -> Workload:
    gen = _gen(device, seed)
    x, codes = _normal_binned(rows, 28, 64, gen, device)
    w = torch.randn(28, generator=gen, device=device)
    noise = 0.5 * torch.randn(rows, generator=gen, device=device)
    y = ((x @ w + noise) > 0).float()
    return Workload("tiny", codes, 64, y, dict(bits=2, objective=0, num_leaves=31, num_trees=10,
                                                 learning_rate=0.1, min_data_in_leaf=20))


def tall(device="cpu", rows=1_000_000, seed=MASTER_SEED + 2) -> Workload:
    gen = _gen(device, seed)
    x, codes = _normal_binned(rows, 28, 255, gen, device)
    # a random complete depth-6 tree over the features: 63 (feature, threshold) nodes, 64 leaf labels
    feat = torch.randint(0, 28, (63,), generator=gen, device=device)
    thr = torch.randn(63, generator=gen, device=device) * 0.7
    leaf_label = torch.randint(0, 2, (64,), generator=gen, device=device).float()
    node = torch.zeros(rows, dtype=torch.long, device=device)
    for _ in range(6):
        go_right = x.gather(1, feat[node].unsqueeze(1)).squeeze(1) > thr[node]
        node = 2 * node + 1 + go_right.long()
    y = leaf_label[node - 63]
    flip = torch.rand(rows, generator=gen, device=device) < 0.10
    y = torch.where(flip, 1.0 - y, y)
    return Workload("tall", codes, 255, y, dict(bits=3, objective=0, num_leaves=255, num_trees=100,
                                                  learning_rate=0.1, min_data_in_leaf=20))


def wide(device="cpu", rows=400_000, features=2000, seed=MASTER_SEED + 3) -> Workload:
    gen = _gen(device, seed)
    w = torch.randn(features, generator=gen, device=device)
    w = w * (torch.rand(features, generator=gen, device=device) < 0.05).float()
    codes = torch.empty((rows, features), dtype=torch.uint8, device=device)
    logit = torch.zeros(rows, device=device)
    for j0 in range(0, features, 50):
        j1 = min(features, j0 + 50)
        x = torch.randn((rows, j1 - j0), generator=gen, device=device)
        codes[:, j0:j1] = quantile_bin(x, 255)
        logit += x @ w[j0:j1]
    y = ((logit + torch.randn(rows, generator=gen, device=device)) > 0).float()
    return Workload("wide", codes, 255, y, dict(bits=3, objective=0, num_leaves=255, num_trees=100,
                                                  learning_rate=0.1, min_data_in_leaf=20))


def large(device="cpu", rows=10_500_000, seed=MASTER_SEED + 4) -> Workload:
    gen = _gen(device, seed)
    codes = torch.empty((rows, 28), dtype=torch.uint8, device=device)
    step_feat = torch.randint(0, 28, (8,), generator=gen, device=device)
    step_thr = torch.randn(8, generator=gen, device=device) * 0.8
    step_height = torch.randn(8, generator=gen, device=device)
    y = 0.1 * torch.randn(rows, generator=gen, device=device)
    for j in range(28):
        x = torch.randn((rows, 1), generator=gen, device=device)
        codes[:, j:j + 1] = quantile_bin(x, 255)
        for k in range(8):
            if int(step_feat[k]) == j:
                y += step_height[k] * (x[:, 0] > step_thr[k]).float()
    return Workload("large", codes, 255, y, dict(bits=4, objective=1, num_leaves=255, num_trees=500,
                                                   learning_rate=0.1, min_data_in_leaf=20))


def sweep_bins(rows, features, n_bins, device="cpu", seed=MASTER_SEED + 5) -> torch.Tensor:
    """Uniform codes on [0, n_bins); for the odd-numbered features 90% of the entries are bin 0."""
    gen = _gen(device, seed + 1000003 * features + 7919 * n_bins)
    codes = torch.empty((rows, features), dtype=torch.uint8, device=device)
    step = max(1, (1 << 28) // max(rows, 1))
    odd = (torch.arange(features, device=device) % 2 == 1)
    for j0 in range(0, features, step):
        j1 = min(features, j0 + step)
        c = torch.randint(0, n_bins, (rows, j1 - j0), generator=gen, device=device, dtype=torch.uint8)
        keep = torch.rand((rows, j1 - j0), generator=gen, device=device) >= 0.9
        c = torch.where(odd[j0:j1].unsqueeze(0) & ~keep, torch.zeros_like(c), c)
        codes[:, j0:j1] = c
    return codes


def sweep_gradients(rows, device="cpu", seed=MASTER_SEED + 6):
    """Logistic-loss gradients of N(0,1) logits against Bernoulli(1/2) labels: (g, h) float32."""
    gen = _gen(device, seed)
    s = torch.randn(rows, generator=gen, device=device)
    y = (torch.rand(rows, generator=gen, device=device) < 0.5).float()
    p = torch.sigmoid(s)
    return (p - y).contiguous(), (p * (1 - p)).contiguous()


def subset_rows(rows, device="cpu", seed=MASTER_SEED + 7, frac=0.5) -> torch.Tensor:
    """Ascending row indices of a Bernoulli(frac) subset, as int32 holding uint32 values."""
    gen = _gen(device, seed)
    mask = torch.rand(rows, generator=gen, device=device) < frac
    return torch.nonzero(mask).squeeze(1).to(torch.int32)


CONFIGS = {"tiny": tiny, "tall": tall, "wide": wide, "large": large}
