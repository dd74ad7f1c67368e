"""Seeded synthetic inputs shaped like the paper's node-classification workloads.

The paper's datasets (citation networks, Reddit, OGBN-Products) are not available, so
graphs, features and weights are drawn here with the same sizes, sparsity and degree
skew.  This module holds no arithmetic of the method itself: it only produces arrays
that the tests hand unchanged to the CPU oracle and to the CUDA library alike.

Arrays are built with torch tensor ops on a chosen device (the large graphs take minutes
on a CPU and well under a second on a GPU).  Random bits come from one counter-based
generator, the splitmix64 output function applied to (seed, stream, index), evaluated in
int64 tensor arithmetic, so the integer streams are identical on every device; the float
transforms on top of them (pow, log, cos, cumsum) may differ in the last place between
devices, which is harmless because a workload is drawn once and then copied to whoever
needs it.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    seed: int
    n: int                      # nodes
    e_dir: int                  # directed edges (both directions counted, no self-loops)
    dims: tuple                 # d_0 (features), hidden..., classes
    features: str               # "bernoulli" | "tfidf" | "normal"
    density: float = 1.0        # share of non-zero feature entries
    bn_every_layer: bool = False  # batch-norm constants before every layer (else input only)
    gamma: float = 2.3          # power-law exponent of the target degrees
    kmax_over_mean: float = 50.0


# Shapes of the five benchmark configurations (nodes, directed edges, widths).
WORKLOADS: Dict[str, WorkloadSpec] = {
    "c1": WorkloadSpec("c1", 1001, 2_708, 10_556, (1433, 64, 7), "bernoulli", 0.013),
    "c2": WorkloadSpec("c2", 1002, 3_327, 9_104, (3703, 64, 6), "bernoulli", 0.0085),
    "c3": WorkloadSpec("c3", 1003, 19_717, 88_648, (500, 64, 3), "tfidf", 0.10),
    "c4": WorkloadSpec("c4", 1004, 232_965, 114_600_000, (602, 256, 41), "normal"),
    "c5": WorkloadSpec("c5", 1005, 2_449_029, 123_700_000, (100, 256, 256, 47), "normal",
                       bn_every_layer=True),
}


def _i64(x: int) -> int:
    """Two's-complement int64 value of an unsigned 64-bit constant."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _i64(0x9E3779B97F4A7C15)
_M1 = _i64(0xBF58476D1CE4E5B9)
_M2 = _i64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 lanes."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def random_bits(seed: int, stream: int, count: int, device, offset: int = 0) -> torch.Tensor:
    """int64 tensor of ``count`` 64-bit words: splitmix64's output function of a per-stream
    base plus (index + 1) times the golden-ratio increment (wrapping int64 arithmetic)."""
    base = _i64((int(seed) * 0x2545F4914F6CDD1D + int(stream) * 0xD1342543DE82EF95) & ((1 << 64) - 1))
    i = torch.arange(offset + 1, offset + count + 1, dtype=torch.int64, device=device)
    z = i * _GOLDEN + base
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def uniform(seed: int, stream: int, count: int, device, offset: int = 0) -> torch.Tensor:
    """float64 in [0, 1): the top 53 bits of each word."""
    return _lsr(random_bits(seed, stream, count, device, offset), 11).to(torch.float64) * (2.0 ** -53)


def normal(seed: int, stream: int, count: int, device) -> torch.Tensor:
    """float32 N(0,1) by the Box-Muller transform of two uniform streams."""
    out = torch.empty(count, dtype=torch.float32, device=device)
    step = 1 << 25
    for a in range(0, count, step):
        m = min(step, count - a)
        u1 = uniform(seed, stream, m, device, a)
        u2 = uniform(seed, stream + 1000, m, device, a)
        r = torch.sqrt(-2.0 * torch.log1p(-u1))
        out[a:a + m] = (r * torch.cos(2.0 * np.pi * u2)).to(torch.float32)
    return out


def power_law_graph(n: int, e_dir: int, seed: int, gamma: float = 2.3,
                    kmax_over_mean: float = 50.0, device="cpu"):
    """Undirected Chung-Lu style graph with power-law target degrees.

    Returns (rowptr int64 [n+1], colidx int32 [e]) of the symmetric adjacency A without
    self-loops: every undirected edge appears in both directions, columns ascending in a
    row, no repeats.  Node ids carry no locality (target degrees are i.i.d. over ids), which
    is the worst case for the neighbour gathers.  The number of directed edges is e_dir
    rounded down to an even number, or fewer when the graph cannot hold that many pairs.
    """
    n = int(n)
    want = int(e_dir) // 2
    if n < 2 or want <= 0:
        return (torch.zeros(n + 1, dtype=torch.int64, device=device),
                torch.zeros(0, dtype=torch.int32, device=device))
    want = min(want, n * (n - 1) // 2)
    mean = 2.0 * want / n
    k = (1.0 - uniform(seed, 10, n, device)) ** (-1.0 / (gamma - 1.0))   # Pareto, k_min = 1
    k = torch.clamp(k, max=float(kmax_over_mean * k.mean()))              # truncated tail
    k = k * (mean / float(k.mean()))
    k = torch.clamp(k, max=float(n - 1))
    cdf = torch.cumsum(k, 0)
    cdf = cdf / cdf[-1]
    keys = torch.zeros(0, dtype=torch.int64, device=device)
    draw, drawn = want, 0
    for _ in range(64):
        m = int(draw * 1.1) + 16
        a = torch.searchsorted(cdf, uniform(seed, 11, m, device, drawn)).clamp_(max=n - 1)
        b = torch.searchsorted(cdf, uniform(seed, 12, m, device, drawn)).clamp_(max=n - 1)
        drawn += m
        keep = a != b
        lo = torch.minimum(a, b)[keep]
        hi = torch.maximum(a, b)[keep]
        keys = torch.unique(torch.cat([keys, lo * n + hi]))
        if keys.shape[0] >= want:
            break
        draw = max(want - keys.shape[0], 1024)
    if keys.shape[0] > want:                       # thin the sorted pair list evenly
        have = keys.shape[0]
        pick = (torch.arange(want, dtype=torch.float64, device=device) * (have / want)).to(torch.int64)
        keys = keys[pick.clamp_(max=have - 1)]
    lo = keys // n
    hi = keys % n
    both, _ = torch.sort(torch.cat([lo * n + hi, hi * n + lo]))
    src = both // n
    dst = (both % n).to(torch.int32)
    rowptr = torch.zeros(n + 1, dtype=torch.int64, device=device)
    rowptr[1:] = torch.cumsum(torch.bincount(src, minlength=n), 0)
    return rowptr, dst


def edge_list(rowptr: torch.Tensor, colidx: torch.Tensor):
    """(src, dst) int32 numpy arrays of a CSR adjacency."""
    rp = rowptr.cpu().numpy()
    n = rp.shape[0] - 1
    src = np.repeat(np.arange(n, dtype=np.int32), np.diff(rp))
    return src, colidx.cpu().numpy().astype(np.int32, copy=False)


def features(kind: str, n: int, d: int, seed: int, density: float = 1.0, device="cpu") -> torch.Tensor:
    """fp32 [n, d] row-major: 0/1 bag-of-words, TF-IDF-like non-negative, or N(0,1)."""
    cnt = n * d
    if kind == "bernoulli":
        x = (uniform(seed, 20, cnt, device) < density).to(torch.float32)
    elif kind == "tfidf":
        mask = uniform(seed, 20, cnt, device) < density
        vals = torch.exp(normal(seed, 21, cnt, device) - 3.0)           # log-normal(-3, 1)
        x = torch.where(mask, vals, torch.zeros_like(vals))
    elif kind == "normal":
        x = normal(seed, 21, cnt, device)
    else:
        raise ValueError(kind)
    return x.reshape(n, d).contiguous()


def weights(dims, seed: int, device="cpu") -> List[torch.Tensor]:
    """fp32 [d_in, d_out] per layer, N(0, 1/fan_in)."""
    out = []
    for l, (d_in, d_out) in enumerate(zip(dims[:-1], dims[1:])):
        w = normal(seed, 30 + 2 * l, d_in * d_out, device) * float(d_in ** -0.5)
        out.append(w.reshape(d_in, d_out).contiguous())
    return out


@dataclass
class Workload:
    spec: WorkloadSpec
    rowptr: torch.Tensor        # int64 [n+1]; CSR of A (symmetric, no self-loops)
    colidx: torch.Tensor        # int32 [e]
    X: torch.Tensor             # fp32 [n, d_0]
    W: List[torch.Tensor]       # fp32 [d_in, d_out] per layer

    @property
    def n(self) -> int:
        return self.spec.n

    @property
    def n_layers(self) -> int:
        return len(self.spec.dims) - 1

    def bn_layers(self) -> List[bool]:
        """Which layers have batch-norm constants on their input (Sec. 7 setups: the input
        features only on the citation-style workloads, every layer on the OGB-style one)."""
        return [l == 0 or self.spec.bn_every_layer for l in range(self.n_layers)]


def scaled_spec(spec: WorkloadSpec, scale: float) -> WorkloadSpec:
    """Shrink nodes and edges together (same mean degree)."""
    n = max(2, int(spec.n * scale))
    e = int(spec.e_dir * scale) // 2 * 2
    return WorkloadSpec("%s@%g" % (spec.name, scale), spec.seed, n, e, spec.dims, spec.features,
                        spec.density, spec.bn_every_layer, spec.gamma, spec.kmax_over_mean)


def make_workload(name_or_spec, scale: Optional[float] = None, device="cpu") -> Workload:
    spec = WORKLOADS[name_or_spec] if isinstance(name_or_spec, str) else name_or_spec
    if scale is not None and scale != 1.0:
        spec = scaled_spec(spec, scale)
    rowptr, colidx = power_law_graph(spec.n, spec.e_dir, spec.seed, spec.gamma,
                                     spec.kmax_over_mean, device)
    X = features(spec.features, spec.n, spec.dims[0], spec.seed, spec.density, device)
    W = weights(spec.dims, spec.seed, device)
    return Workload(spec, rowptr, colidx, X, W)
