"""Seeded synthetic attention inputs: phi(Q), phi(K) = ReLU(N(0,1)) drawn directly in R^m
(the paper's feature map is ReLU, Table 2) and V ~ N(0,1).  Input generation only."""
from __future__ import annotations

import numpy as np
import torch


def to_dtype(x: np.ndarray, dtype: str) -> torch.Tensor:
    """fp32 numpy array -> CPU torch tensor of the workload's storage type."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    if dtype == "bf16":
        return t.to(torch.bfloat16)
    if dtype == "fp32":
        return t
    raise ValueError(dtype)


def widen(t: torch.Tensor) -> np.ndarray:
    """Storage-type tensor -> fp32 numpy holding exactly the same values."""
    return t.detach().to("cpu").to(torch.float32).numpy()


def qkv(G: int, N: int, m: int, d: int, dtype: str, seed: int):
    """Returns (phiQ [G,N,m], phiK [G,N,m], V [G,N,d]) as CPU torch tensors of `dtype`."""
    rng = np.random.default_rng(seed)
    q = np.maximum(rng.standard_normal((G, N, m), dtype=np.float32), 0.0)
    k = np.maximum(rng.standard_normal((G, N, m), dtype=np.float32), 0.0)
    v = rng.standard_normal((G, N, d), dtype=np.float32)
    return to_dtype(q, dtype), to_dtype(k, dtype), to_dtype(v, dtype)
