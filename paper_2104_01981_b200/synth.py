"""Seeded synthetic gradients and the tensor-shape lists of the five benchmark workloads.

This module serves both the CUDA path and the CPU oracle with the *same input bytes*; it
holds none of the method's arithmetic (no fold, no selection, no decode).  Everything is
drawn from a ``torch.Generator`` seeded from (seed0, config, worker, step), so a run is
reproducible on a given device type.  Real training gradients are not available offline;
these stand in for them with the sizes, per-layer structure and value distributions the
workload definitions name (Gaussian with 1/sqrt(fan_in) scale, Student-t with 3 degrees of
freedom, Gaussian with rare 50-sigma outliers).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Tuple

import torch

SEED0 = 1234


# --------------------------------------------------------------------------- shapes
def resnet50_shapes() -> List[Tuple[int, ...]]:
    """The 161 parameter tensors of the standard ResNet-50, in module order."""
    shapes: List[Tuple[int, ...]] = [(64, 3, 7, 7), (64,), (64,)]
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            shapes += [(planes, inplanes, 1, 1), (planes,), (planes,)]
            shapes += [(planes, planes, 3, 3), (planes,), (planes,)]
            shapes += [(planes * 4, planes, 1, 1), (planes * 4,), (planes * 4,)]
            if b == 0:
                shapes += [(planes * 4, inplanes, 1, 1), (planes * 4,), (planes * 4,)]
            inplanes = planes * 4
    shapes += [(1000, 2048), (1000,)]
    return shapes


def bert_base_shapes() -> List[Tuple[int, ...]]:
    """BERT-base parameter shapes (embeddings, 12 encoder layers, pooler)."""
    d, ff = 768, 3072
    shapes: List[Tuple[int, ...]] = [(30522, d), (512, d), (2, d), (d,), (d,)]
    for _ in range(12):
        for _ in range(4):                       # Q, K, V, attention output
            shapes += [(d, d), (d,)]
        shapes += [(d,), (d,)]                   # LayerNorm
        shapes += [(ff, d), (ff,), (d, ff), (d,)]
        shapes += [(d,), (d,)]                   # LayerNorm
    shapes += [(d, d), (d,)]                     # pooler
    return shapes


def gpt2_medium_shapes() -> List[Tuple[int, ...]]:
    """GPT-2-medium parameter shapes (24 layers, d=1024, vocabulary 50257)."""
    d = 1024
    shapes: List[Tuple[int, ...]] = [(50257, d), (1024, d)]
    for _ in range(24):
        shapes += [(d,), (d,), (d, 3 * d), (3 * d,), (d, d), (d,)]
        shapes += [(d,), (d,), (d, 4 * d), (4 * d,), (4 * d, d), (d,)]
    shapes += [(d,), (d,)]
    return shapes


def numel(shape: Tuple[int, ...]) -> int:
    return int(math.prod(shape))


def fan_in(shape: Tuple[int, ...]) -> int:
    """in_channels*kh*kw for convolutions, in_features for linear weights, numel for 1-D."""
    if len(shape) == 1:
        return shape[0]
    return numel(shape[1:])


# --------------------------------------------------------------------------- workloads
@dataclass
class Workload:
    """One benchmark configuration: tensor sizes, density, worker count, step count."""
    name: str
    config_id: int
    sizes: List[int]                 # elements per tensor of the concatenated flat gradient
    density: float
    workers: int
    steps: int
    dist: str                        # "normal" | "layer_normal" | "student_t3" | "normal_outliers"
    scales: List[float] = field(default_factory=list)   # per-tensor sigma ("layer_normal")
    sigma: float = 1.0

    @property
    def total_n(self) -> int:
        return sum(self.sizes)


def workload(config_id: int) -> Workload:
    """Workloads 0..4 are the five configurations, in the order they are listed."""
    if config_id == 0:
        return Workload("c1_single_1m_normal", 0, [1 << 20], 0.01, 1, 3, "normal", sigma=1.0)
    if config_id in (1, 3):
        shp = resnet50_shapes()
        w = Workload("c2_resnet50_layerwise" if config_id == 1 else "c4_resnet50_8workers",
                     config_id, [numel(s) for s in shp], 0.001,
                     1 if config_id == 1 else 8, 10 if config_id == 1 else 1, "layer_normal",
                     scales=[1.0 / math.sqrt(fan_in(s)) for s in shp])
        return w
    if config_id == 2:
        n = sum(numel(s) for s in bert_base_shapes())
        return Workload("c3_bert_base_110m_student_t", 2, [n], 0.01, 1, 10, "student_t3", sigma=0.02)
    if config_id == 4:
        n = sum(numel(s) for s in gpt2_medium_shapes())
        return Workload("c5_gpt2_medium_355m_outliers", 4, [n], 0.001, 16, 5, "normal_outliers",
                        sigma=0.02)
    raise ValueError(f"unknown config {config_id}")


# --------------------------------------------------------------------------- generators
def _seed(config_id: int, worker: int, step: int, seed0: int = SEED0) -> int:
    """A fixed mix of (seed0, config, worker, step); any injective-enough hash will do."""
    x = (seed0 * 1000003 + config_id) * 1000003 + worker
    x = (x * 1000003 + step) & 0x7FFFFFFFFFFFFFFF
    return x


def gradient(w: Workload, worker: int, step: int, device: str | torch.device = "cpu",
             out: torch.Tensor | None = None, seed0: int = SEED0) -> torch.Tensor:
    """Flat fp32 gradient of ``w.total_n`` elements for (worker, step), on ``device``.

    Generated chunk-wise so that the transient memory stays a small multiple of one chunk.
    """
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(_seed(w.config_id, worker, step, seed0))
    n = w.total_n
    g = out if out is not None else torch.empty(n, dtype=torch.float32, device=device)
    assert g.numel() == n and g.dtype == torch.float32
    if w.dist == "layer_normal":
        off = 0
        for sz, sc in zip(w.sizes, w.scales):
            g[off:off + sz].normal_(0.0, 1.0, generator=gen).mul_(sc)
            off += sz
        return g
    chunk = 1 << 24
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        v = g[lo:hi]
        if w.dist == "normal":
            v.normal_(0.0, w.sigma, generator=gen)
        elif w.dist == "student_t3":
            # t_3 = Z / sqrt(chi2_3 / 3), chi2_3 = sum of three squared standard normals
            v.normal_(0.0, 1.0, generator=gen)
            chi = torch.zeros_like(v)
            tmp = torch.empty_like(v)
            for _ in range(3):
                tmp.normal_(0.0, 1.0, generator=gen)
                chi.addcmul_(tmp, tmp)
            v.div_(chi.div_(3.0).sqrt_()).mul_(w.sigma)
        elif w.dist == "normal_outliers":
            # N(0, sigma^2); each element independently replaced, with probability 1e-4,
            # by +-50 sigma exactly (random sign)
            v.normal_(0.0, w.sigma, generator=gen)
            u = torch.empty_like(v).uniform_(0.0, 1.0, generator=gen)
            sgn = torch.empty_like(v).uniform_(0.0, 1.0, generator=gen)
            spike = torch.where(sgn < 0.5, -50.0 * w.sigma, 50.0 * w.sigma).to(torch.float32)
            torch.where(u < 1e-4, spike, v, out=v)
        else:
            raise ValueError(w.dist)
    return g


def quantised_gradient(n: int, seed: int, step: float = 0.125,
                       device: str | torch.device = "cpu") -> torch.Tensor:
    """Tie-stress input: N(0,1) rounded to multiples of ``step`` so that thousands of equal
    magnitudes straddle the k-th largest."""
    gen = torch.Generator(device=torch.device(device))
    gen.manual_seed(seed)
    g = torch.empty(n, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
    return torch.round(g / step) * step


# --------------------------------------------------------------------------- sparse sets
def _distinct_sorted(rng, n: int, k: int):
    """k distinct integers of [0, n), ascending (numpy, no permutation of n)."""
    import numpy as np
    if k >= n:
        return np.arange(n, dtype=np.int64)
    if k > n // 2:
        drop = _distinct_sorted(rng, n, n - k)
        keep = np.ones(n, dtype=bool)
        keep[drop] = False
        return np.nonzero(keep)[0]
    got = np.unique(rng.integers(0, n, size=int(k * 1.1) + 16))
    while got.size < k:
        got = np.unique(np.concatenate([got, rng.integers(0, n, size=k - got.size + 16)]))
    if got.size > k:
        got = np.sort(rng.choice(got, size=k, replace=False))
    return got


def sparse_set(sizes, ks, seed: int, scale: float = 1.0):
    """A seeded sparse set laid out like a top-k output: for every tensor t, ks[t] distinct flat
    indices inside the tensor, ascending, with N(0, scale^2) values.  Returns numpy arrays
    (uint32 indices, float32 values).  Input generator only: nothing here selects anything."""
    import numpy as np
    rng = np.random.default_rng(seed)
    idx, off = [], 0
    for n, k in zip(sizes, ks):
        idx.append(_distinct_sorted(rng, int(n), int(k)) + off)
        off += int(n)
    idx = np.concatenate(idx).astype(np.uint32) if idx else np.zeros(0, np.uint32)
    val = (rng.standard_normal(idx.size) * scale).astype(np.float32)
    return idx, val


# --------------------------------------------------------------------------- embedding-table batches
def ecrm_tables(n_rows: int, dim: int, k: int, seed: int, device: str | torch.device = "cpu",
                integer_valued: bool = False):
    """k embedding-table shards [n_rows][dim] with N(0, 0.01^2)-like entries (or small integers,
    for cases that must be exact) and zero optimizer state.  Input generator only."""
    gen = torch.Generator(device=torch.device(device))
    gen.manual_seed(seed)
    shards = []
    for _ in range(k):
        e = torch.empty(n_rows, dim, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
        shards.append(torch.round(e * 8.0) if integer_valued else e * 0.01)
    return shards


def ecrm_batch(n_rows: int, m: int, dim: int, seed: int, device: str | torch.device = "cpu",
               integer_valued: bool = False):
    """One batch's aggregated sparse gradient for a shard: m distinct row numbers (random order,
    as a hash-based unique leaves them) and their gradient rows."""
    import numpy as np
    rng = np.random.default_rng(seed)
    rows = _distinct_sorted(rng, n_rows, m)
    rng.shuffle(rows)
    gen = torch.Generator(device=torch.device(device))
    gen.manual_seed(seed + 17)
    g = torch.empty(m, dim, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
    g = torch.round(g * 4.0) if integer_valued else g * 0.05
    return torch.from_numpy(rows.astype(np.uint32).view(np.int32)).to(device), g
