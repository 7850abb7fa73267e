"""Seeded synthetic inputs: graph generators and the named workload shapes.

This module holds NO arithmetic of the walk / SGNS method.  It only produces
input data (CSR graphs, degree weights, start nodes) that both the CUDA library
and the CPU oracle receive as plain arrays, and the table of workload shapes.

The graphs stand in for the public graphs the paper trains on (Section 4
"Datasets": Reddit, ogbn-products, ogbn-papers100M): power-law degrees,
10^4..10^8 nodes, average degree 10..20.

Randomness comes from a counter hash (splitmix64 of seed and element index)
evaluated with wrapping int64 tensor arithmetic, so a generator is a pure
function of (seed, sizes) and runs unchanged on CPU or CUDA tensors.  The two
devices may still differ in the last bit of floating-point `pow`, so a graph is
always generated once and handed to every consumer as data.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

_MASK32 = 0xFFFFFFFF


def _wrap(x: int) -> int:
    """Two's-complement int64 value of an unsigned 64-bit constant."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _wrap(0x9E3779B97F4A7C15)
_M1 = _wrap(0xBF58476D1CE4E5B9)
_M2 = _wrap(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def hash64(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser of (seed, stream, idx); int64 bit patterns."""
    z = idx * _GOLDEN + _wrap(seed * 0xD1342543DE82EF95 + stream * 0xA0761D6478BD642F + 1)
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def uniform01(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """float64 uniforms in [0, 1) with 53 random bits."""
    return _lsr(hash64(seed, stream, idx), 11).to(torch.float64) * (1.0 / 9007199254740992.0)


@dataclass
class CSRGraph:
    """CSR with strictly increasing rows.  offsets int32 or int64, cols int32."""
    n_nodes: int
    offsets: torch.Tensor
    cols: torch.Tensor

    @property
    def n_edges(self) -> int:
        return int(self.cols.numel())

    def degrees(self) -> torch.Tensor:
        return (self.offsets[1:] - self.offsets[:-1]).to(torch.int64)

    def to(self, device) -> "CSRGraph":
        return CSRGraph(self.n_nodes, self.offsets.to(device), self.cols.to(device))


def _relabel_params(n: int, seed: int):
    """Multiplier a (coprime with n) and shift b of the id bijection v -> (a v + b) mod n."""
    a = (0x9E3779B97F4A7C15 ^ (seed * 0x2545F4914F6CDD1D)) % n
    a = max(a, 1)
    while math.gcd(a, n) != 1:
        a += 1
    b = (seed * 0x632BE59BD9B4E019 + 12345) % n
    return a, b


def _csr_from_directed(src: torch.Tensor, dst: torch.Tensor, n: int, offsets64: bool) -> CSRGraph:
    """Sort (src, dst), drop duplicates, build CSR.  src/dst int64."""
    keys = torch.unique((src << 32) | dst)           # sorted, duplicates removed
    del src, dst
    rows = keys >> 32
    cols = (keys & _MASK32).to(torch.int32)
    del keys
    counts = torch.bincount(rows, minlength=n)
    del rows
    off = torch.zeros(n + 1, dtype=torch.int64, device=cols.device)
    torch.cumsum(counts, 0, out=off[1:])
    if not offsets64:
        assert int(off[-1]) < 2 ** 31
        off = off.to(torch.int32)
    return CSRGraph(n, off, cols)


def chung_lu_cutoff(n: int, avg_degree: float, exponent: float):
    """Scale c and shift i0 of the expected-degree sequence w_i = c (i + i0)^(-a).

    a = 1/(exponent-1); c makes the (continuous) mean equal avg_degree; i0 is the
    smallest shift >= 1 for which the largest weight stays below sqrt(sum of
    weights), the structural cutoff that keeps edge probabilities below one.
    """
    a = 1.0 / (exponent - 1.0)
    total = n * avg_degree

    def scale(i0):
        integral = ((n + i0) ** (1 - a) - i0 ** (1 - a)) / (1 - a)
        return total / integral

    lo, hi = 1.0, float(n)
    if scale(lo) * lo ** (-a) <= math.sqrt(total):
        return scale(lo), lo, a
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if scale(mid) * mid ** (-a) <= math.sqrt(total):
            hi = mid
        else:
            lo = mid
    return scale(hi), hi, a


def chung_lu_graph(n: int, avg_degree: float, exponent: float, seed: int,
                   device="cpu", offsets64: bool = False, chunk: int = 1 << 26) -> CSRGraph:
    """Undirected Chung-Lu power-law graph as a symmetric CSR.

    n*avg_degree/2 edge draws; both endpoints i.i.d. with probability
    proportional to w_i (inverse of the continuous CDF); self-loops dropped;
    both directions stored; duplicates removed; node ids passed through a
    fixed bijection so that hubs are spread over the id range.
    """
    _, i0, a = chung_lu_cutoff(n, avg_degree, exponent)
    m = int(n * avg_degree / 2)
    e = 1.0 - a
    lo_p, hi_p = i0 ** e, (n + i0) ** e
    ra, rb = _relabel_params(n, seed)
    parts = []
    for start in range(0, m, chunk):
        idx = torch.arange(start, min(m, start + chunk), dtype=torch.int64, device=device)
        ends = []
        for stream in (1, 2):
            u = uniform01(seed, stream, idx)
            x = (lo_p + u * (hi_p - lo_p)) ** (1.0 / e) - i0
            v = x.floor().to(torch.int64).clamp_(0, n - 1)
            ends.append((v * ra + rb) % n)
        keep = ends[0] != ends[1]
        parts.append((ends[0][keep], ends[1][keep]))
    s = torch.cat([p[0] for p in parts])
    t = torch.cat([p[1] for p in parts])
    del parts
    src = torch.cat([s, t])
    dst = torch.cat([t, s])
    del s, t
    return _csr_from_directed(src, dst, n, offsets64)


def rmat_graph(n: int, n_edges: int, abcd=(0.57, 0.19, 0.19, 0.05), seed: int = 0,
               device="cpu", offsets64: bool = True, chunk: int = 1 << 26) -> CSRGraph:
    """Directed R-MAT graph: recursive quadrant choice on a 2^scale grid.

    Draws edges until n_edges of them have both endpoints below n (the grid is
    the next power of two), drops self-loops and duplicates, keeps directions.
    """
    scale = max(1, (n - 1).bit_length())
    a, b, c, _ = abcd
    ra, rb = _relabel_params(n, seed)
    srcs, dsts, have, start = [], [], 0, 0
    while have < n_edges:
        idx = torch.arange(start, start + chunk, dtype=torch.int64, device=device)
        start += chunk
        src = torch.zeros_like(idx)
        dst = torch.zeros_like(idx)
        for level in range(scale):
            u = uniform01(seed, 16 + level, idx)
            right = ((u >= a) & (u < a + b)) | (u >= a + b + c)      # quadrants b, d
            down = u >= a + b                                         # quadrants c, d
            src = (src << 1) | down.to(torch.int64)
            dst = (dst << 1) | right.to(torch.int64)
        keep = (src < n) & (dst < n)
        src, dst = src[keep], dst[keep]
        take = min(int(src.numel()), n_edges - have)
        srcs.append(src[:take])
        dsts.append(dst[:take])
        have += take
    src = torch.cat(srcs)
    dst = torch.cat(dsts)
    del srcs, dsts
    keep = src != dst
    src = (src[keep] * ra + rb) % n
    dst = (dst[keep] * ra + rb) % n
    return _csr_from_directed(src, dst, n, offsets64)


def ring_with_chords(n: int, device="cpu") -> CSRGraph:
    """Small connected, non-bipartite, undirected test graph: cycle + a few chords."""
    v = torch.arange(n, dtype=torch.int64, device=device)
    src = [v, (v + 1) % n]
    dst = [(v + 1) % n, v]
    ch = v[v % 3 == 0]
    src += [ch, (ch + 2) % n]
    dst += [(ch + 2) % n, ch]
    return _csr_from_directed(torch.cat(src), torch.cat(dst), n, False)


@dataclass(frozen=True)
class Workload:
    """Shape of one named configuration (graph recipe + walk + SGNS parameters)."""
    name: str
    graph: str            # "chung_lu" | "rmat"
    n_nodes: int
    avg_degree: float
    exponent: float
    graph_seed: int
    offsets64: bool
    walk_kind: str        # "uniform" | "node2vec"
    walks_per_node: int
    walk_len: int
    window: int
    n_neg: int
    dim: int
    lr0: float
    lr_schedule: str      # "constant" | "linear"
    p: float = 1.0
    q: float = 1.0
    n_edges_target: int = 0
    forward_only: bool = False   # pairs (i, j) with j > i only: LINE's (source, neighbour) edges

    def make_graph(self, device="cpu", scale: float = 1.0) -> CSRGraph:
        """Generate the graph; scale < 1 shrinks the node count (same recipe)."""
        n = max(16, int(self.n_nodes * scale))
        if self.graph == "chung_lu":
            return chung_lu_graph(n, self.avg_degree, self.exponent, self.graph_seed,
                                  device=device, offsets64=self.offsets64)
        return rmat_graph(n, max(16, int(self.n_edges_target * scale)),
                          seed=self.graph_seed, device=device, offsets64=self.offsets64)


WORKLOADS = {
    "tiny_deepwalk": Workload("tiny_deepwalk", "chung_lu", 10_000, 10, 2.5, 0, False,
                              "uniform", 1, 10, 5, 5, 64, 0.025, "linear"),
    "deepwalk_medium": Workload("deepwalk_medium", "chung_lu", 1_000_000, 20, 2.1, 1, False,
                                "uniform", 10, 40, 10, 5, 128, 0.025, "constant"),
    "node2vec_4m": Workload("node2vec_4m", "chung_lu", 4_000_000, 16, 2.3, 2, False,
                            "node2vec", 10, 80, 10, 5, 128, 0.025, "constant", p=0.5, q=2.0),
    # LINE (Section 3.2 / Section 4: a source, one positive and 5 negatives per source node): each
    # "walk" is one sampled edge; the paper's lr 1.0 belongs to its mean-reduced loss, the summed
    # per-pair update here keeps the word2vec-scale 0.025
    "line_medium": Workload("line_medium", "chung_lu", 1_000_000, 20, 2.1, 1, False,
                            "uniform", 20, 2, 1, 5, 128, 0.025, "constant", forward_only=True),
    "deepwalk_large": Workload("deepwalk_large", "chung_lu", 50_000_000, 16, 2.1, 3, True,
                               "uniform", 4, 40, 5, 5, 128, 0.025, "constant"),
    "rmat_billion": Workload("rmat_billion", "rmat", 100_000_000, 10, 0.0, 4, True,
                             "uniform", 2, 20, 5, 10, 64, 0.025, "constant",
                             n_edges_target=1_000_000_000),
}

