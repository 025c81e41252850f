"""Seeded synthetic graphs, returned as CSR of the weighted adjacency matrix W.

Input generation only: nothing here takes part in the method's arithmetic
(no walks, no features, no attention).  Every generator returns a `Graph`
whose CSR has rows sorted by column index, int32 indices and fp32 weights.
W is symmetric in every generator (the mask M_alpha = sum_k alpha_k W^k is
defined for an undirected graph, Sec. 3 / Eq. 4).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class Graph:
    rowptr: np.ndarray  # int32 [N+1]
    col: np.ndarray     # int32 [E]
    w: np.ndarray       # float32 [E]

    @property
    def N(self) -> int:
        return int(self.rowptr.shape[0] - 1)

    @property
    def E(self) -> int:
        return int(self.col.shape[0])

    def dense(self) -> np.ndarray:
        """Dense fp64 copy of W (tiny graphs only)."""
        W = np.zeros((self.N, self.N), dtype=np.float64)
        for i in range(self.N):
            s, e = self.rowptr[i], self.rowptr[i + 1]
            W[i, self.col[s:e]] = self.w[s:e].astype(np.float64)
        return W


def _csr_from_pairs(N: int, src: np.ndarray, dst: np.ndarray, w: np.ndarray) -> Graph:
    order = np.lexsort((dst, src))
    src, dst, w = src[order], dst[order], w[order]
    counts = np.bincount(src, minlength=N)
    rowptr = np.zeros(N + 1, dtype=np.int64)
    np.cumsum(counts, out=rowptr[1:])
    return Graph(rowptr.astype(np.int32), dst.astype(np.int32), w.astype(np.float32))


def grid_graph(nx: int, ny: int, weight: float, diagonals: bool) -> Graph:
    """nx x ny grid, node id = x*ny + y; 4-neighbour, or 8-neighbour with diagonals."""
    if diagonals:
        offs = [(dx, dy) for dx in (-1, 0, 1) for dy in (-1, 0, 1) if (dx, dy) != (0, 0)]
    else:
        offs = [(1, 0), (-1, 0), (0, 1), (0, -1)]
    xs, ys = np.meshgrid(np.arange(nx), np.arange(ny), indexing="ij")
    xs, ys = xs.ravel(), ys.ravel()
    src, dst = [], []
    for dx, dy in offs:
        X, Y = xs + dx, ys + dy
        ok = (X >= 0) & (X < nx) & (Y >= 0) & (Y < ny)
        src.append((xs * ny + ys)[ok])
        dst.append((X * ny + Y)[ok])
    src, dst = np.concatenate(src), np.concatenate(dst)
    return _csr_from_pairs(nx * ny, src, dst, np.full(src.shape, weight, dtype=np.float32))


def path_graph(N: int, weight: float) -> Graph:
    """1-D grid (the FLOP experiment's topology, Sec. 4 'Time complexity')."""
    i = np.arange(N - 1)
    src = np.concatenate([i, i + 1])
    dst = np.concatenate([i + 1, i])
    return _csr_from_pairs(N, src, dst, np.full(src.shape, weight, dtype=np.float32))


def perfect_matching_graph(N: int, weight: float) -> Graph:
    """N even; node 2a is joined to 2a+1 only, so every degree is 1 and walks are deterministic."""
    assert N % 2 == 0
    i = np.arange(N)
    return _csr_from_pairs(N, i, i ^ 1, np.full(N, weight, dtype=np.float32))


def morton_order(points: np.ndarray, bits: int = 10) -> np.ndarray:
    """Permutation that sorts 3-D points along a Z-order curve (spatial locality of node ids)."""
    lo, hi = points.min(axis=0), points.max(axis=0)
    q = ((points - lo) / np.maximum(hi - lo, 1e-30) * ((1 << bits) - 1)).astype(np.uint64)
    code = np.zeros(points.shape[0], dtype=np.uint64)
    for b in range(bits):
        for a in range(3):
            code |= ((q[:, a] >> np.uint64(b)) & np.uint64(1)) << np.uint64(3 * b + a)
    return np.argsort(code, kind="stable")


def uniform_cube_points(N: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.random((N, 3))


def gaussian_mixture_points(N: int, clusters: int, seed: int) -> np.ndarray:
    """Centres U[0,1]^3, isotropic sigma_c ~ U(0.03, 0.1), equal weights."""
    rng = np.random.default_rng(seed)
    centres = rng.random((clusters, 3))
    sig = rng.uniform(0.03, 0.1, size=clusters)
    which = rng.integers(0, clusters, size=N)
    return centres[which] + rng.standard_normal((N, 3)) * sig[which, None]


def knn_graph(points: np.ndarray, k: int, max_row_sum: float = 0.9, morton: bool = True) -> Graph:
    """Symmetrised kNN graph (edge if either endpoint lists the other), weights
    exp(-dist^2/sigma^2) with sigma the median directed kNN distance, then one
    global scale so that the largest row sum equals `max_row_sum` (keeps W symmetric)."""
    from scipy.spatial import cKDTree

    if morton:
        points = points[morton_order(points)]
    N = points.shape[0]
    dist, idx = cKDTree(points).query(points, k=k + 1)
    dist, idx = dist[:, 1:], idx[:, 1:]
    sigma = float(np.median(dist))
    src = np.repeat(np.arange(N), k)
    dst = idx.ravel()
    d = dist.ravel()
    a = np.minimum(src, dst).astype(np.int64)
    b = np.maximum(src, dst).astype(np.int64)
    code, first = np.unique(a * N + b, return_index=True)
    a, b, d = a[first], b[first], d[first]
    wgt = np.exp(-(d * d) / (sigma * sigma))
    src2 = np.concatenate([a, b])
    dst2 = np.concatenate([b, a])
    w2 = np.concatenate([wgt, wgt])
    rowsum = np.bincount(src2, weights=w2, minlength=N)
    w2 = w2 * (max_row_sum / rowsum.max())
    return _csr_from_pairs(N, src2, dst2, w2)


def random_regular_graph(N: int, seed: int, cycles: int = 4, weight: float | None = None) -> Graph:
    """Simple 2*cycles-regular graph: union of `cycles` random Hamiltonian cycles.
    A cycle edge that repeats an earlier edge is removed by swapping one of its
    endpoints with a random position of the same cycle until no repeat is left."""
    assert N >= 4 * cycles + 2
    rng = np.random.default_rng(seed)
    used = np.empty(0, dtype=np.int64)
    src_all, dst_all = [], []

    def codes(perm):
        nxt = np.roll(perm, -1)
        a, b = np.minimum(perm, nxt), np.maximum(perm, nxt)
        return a.astype(np.int64) * N + b

    for _ in range(cycles):
        perm = rng.permutation(N)
        for _attempt in range(10000):
            c = codes(perm)
            bad = np.isin(c, used)
            # a repeat inside the cycle itself is impossible for N > 2
            if not bad.any():
                break
            pos = np.nonzero(bad)[0]
            other = rng.integers(0, N, size=pos.shape[0])
            for p, o in zip(pos, other):
                perm[p], perm[o] = perm[o], perm[p]
        else:
            raise RuntimeError("could not build a simple regular graph")
        used = np.concatenate([used, codes(perm)])
        nxt = np.roll(perm, -1)
        src_all += [perm, nxt]
        dst_all += [nxt, perm]
    src, dst = np.concatenate(src_all), np.concatenate(dst_all)
    wt = (1.0 / (2 * cycles)) if weight is None else weight
    return _csr_from_pairs(N, src, dst, np.full(src.shape, wt, dtype=np.float32))
