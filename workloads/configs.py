"""The five seeded workloads (graphs, mask coefficients alpha, attention shapes).

They stand in for the paper's workloads: ViT patch grids (Table 2) and the
N = 32768 particle clouds of the point-cloud transformer experiment; none of
the paper's datasets is used.  Input generation only."""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import graphs

GRAPH_SEED = 1234
QKV_SEED = 2024
WALK_SEED = 42
ALPHA_SEED = 7


@dataclass
class Workload:
    name: str
    batch: int
    heads: int
    m: int
    d: int
    dtype: str          # "fp32" | "bf16"
    n_walks: int
    p_halt: float
    max_len: int
    alpha: np.ndarray   # fp64 [max_len+1], mask coefficients alpha_k of Eq. 4
    make_graph: object = field(repr=False, default=None)

    @property
    def G(self) -> int:
        return self.batch * self.heads

    def graph(self) -> graphs.Graph:
        return self.make_graph()


def _alpha_geometric(L: int) -> np.ndarray:
    return 0.5 ** np.arange(L + 1, dtype=np.float64)


def _alpha_uniform(L: int, seed: int) -> np.ndarray:
    """alpha_k ~ U(0,1); alpha_0 is redrawn until it is >= 0.25 (its square root divides the deconvolution)."""
    rng = np.random.default_rng(seed)
    a = rng.random(L + 1)
    while a[0] < 0.25:
        a[0] = rng.random()
    return a


def tiny() -> Workload:
    return Workload("tiny-grid8x8", 1, 1, 16, 16, "fp32", 4, 0.5, 8, _alpha_geometric(8),
                    lambda: graphs.grid_graph(8, 8, 0.25, diagonals=False))


def vit_grid(batch: int = 64, heads: int = 12) -> Workload:
    return Workload("vit-grid14x14", batch, heads, 64, 64, "bf16", 16, 0.1, 10,
                    _alpha_uniform(10, ALPHA_SEED),
                    lambda: graphs.grid_graph(14, 14, 1.0 / 8.0, diagonals=True))


def point_cloud_4096(N: int = 4096) -> Workload:
    return Workload(f"pointcloud-uniform-N{N}", 1, 8, 32, 64, "bf16", 32, 0.1, 12, _alpha_geometric(12),
                    lambda: graphs.knn_graph(graphs.uniform_cube_points(N, GRAPH_SEED), 8))


def point_cloud_32768(N: int = 32768, morton: bool = True) -> Workload:
    return Workload(f"pointcloud-gmm16-N{N}" + ("" if morton else "-unsorted"), 1, 8, 32, 64, "bf16",
                    32, 0.1, 12, _alpha_geometric(12),
                    lambda: graphs.knn_graph(graphs.gaussian_mixture_points(N, 16, GRAPH_SEED), 10,
                                             morton=morton))


def sweep(log2N: int) -> Workload:
    N = 1 << log2N
    return Workload(f"regular8-N2^{log2N}", 1, 4, 32, 64, "bf16", 16, 0.15, 10, _alpha_geometric(10),
                    lambda: graphs.random_regular_graph(N, GRAPH_SEED + log2N))


BY_NAME = {
    "tiny": tiny,
    "vit": vit_grid,
    "pc4096": point_cloud_4096,
    "pc32768": point_cloud_32768,
}
