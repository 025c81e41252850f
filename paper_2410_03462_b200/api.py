"""Object layer over the binding: owns torch device tensors and handles, computes nothing itself."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class Context:
    """A library context on `device`, bound to torch's current stream on that device."""

    def __init__(self, device: int = 0):
        self.device = device
        torch.cuda.set_device(device)
        self.stream = torch.cuda.current_stream(device)
        self.handle = B.grf_ctx_create(device, self.stream.cuda_stream)

    def close(self):
        if self.handle:
            B.grf_ctx_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launches(self) -> int:
        return B.grf_ctx_launch_count(self.handle)


class DeviceGraph:
    """CSR of W resident on the device."""

    def __init__(self, graph, device: int = 0):
        dev = torch.device("cuda", device)
        self.N = graph.N
        self.rowptr = torch.from_numpy(np.ascontiguousarray(graph.rowptr, dtype=np.int32)).to(dev)
        self.col = torch.from_numpy(np.ascontiguousarray(graph.col, dtype=np.int32)).to(dev)
        self.w = torch.from_numpy(np.ascontiguousarray(graph.w, dtype=np.float32)).to(dev)


class Features:
    def __init__(self, ctx: Context, handle: int):
        self.ctx, self.handle = ctx, handle

    def free(self):
        if self.handle:
            B.grf_features_free(self.handle)
            self.handle = None

    def shape(self, which: int):
        rows, cols, nnz, *_ = B.grf_features_view(self.handle, which)
        return rows, cols, nnz

    def to_host(self, which: int):
        """(rowptr, col, val) numpy copies of Phi (0), Psi (1) or Psi^T (2)."""
        rows, cols, nnz = self.shape(which)
        dev = torch.device("cuda", self.ctx.device)
        rp = torch.empty(rows + 1, dtype=torch.int32, device=dev)
        c = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev)
        v = torch.empty(max(nnz, 1), dtype=torch.float32, device=dev)
        B.grf_features_copy(self.ctx.handle, self.handle, which, rp, c, v)
        torch.cuda.synchronize(self.ctx.device)
        return rp.cpu().numpy(), c[:nnz].cpu().numpy(), v[:nnz].cpu().numpy()


def sample(ctx: Context, g: DeviceGraph, seed, n_walks, p_halt, max_len, f_phi, f_psi=None,
           features: Features | None = None) -> Features:
    h = B.grf_sample(ctx.handle, g.N, g.rowptr, g.col, g.w, seed, n_walks, p_halt, max_len, f_phi, f_psi,
                     features.handle if features else None)
    if features:
        features.handle = h
        return features
    return Features(ctx, h)


def features_from_csr(ctx: Context, N, R, phi, psi) -> Features:
    """phi, psi: (rowptr, col, val) numpy triples."""
    dev = torch.device("cuda", ctx.device)

    def up(t):
        rp, c, v = t
        c = np.ascontiguousarray(c, dtype=np.int32); v = np.ascontiguousarray(v, dtype=np.float32)
        if c.size == 0:
            c = np.zeros(1, np.int32); v = np.zeros(1, np.float32)
        return (torch.from_numpy(np.ascontiguousarray(rp, dtype=np.int32)).to(dev),
                torch.from_numpy(c).to(dev), torch.from_numpy(v).to(dev))

    a, b = up(phi), up(psi)
    return Features(ctx, B.grf_features_from_csr(ctx.handle, N, R, *a, *b))


def masked_linear_attn(ctx: Context, feat: Features, phiQ, phiK, V, workspace=None, want_den=False,
                       workspace_bytes=None):
    """phiQ, phiK [G,N,m], V [G,N,d] CUDA tensors (fp32 or bf16).  Returns out, or (out, den)."""
    G, N, m = phiQ.shape
    d = V.shape[2]
    dt = B.dtype_code(phiQ)
    R = feat.shape(0)[1]
    if workspace is None:
        nbytes = workspace_bytes or B.grf_attn_workspace_bytes(G, R, m, d, dt)
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=phiQ.device)
    out = torch.empty_like(V)
    den = torch.empty((G, N), dtype=torch.float32, device=V.device) if want_den else None
    B.grf_masked_linear_attn(ctx.handle, feat.handle, G, N, m, d, dt, phiQ, phiK, V, out, den, workspace,
                             workspace.numel())
    return (out, den) if want_den else out


def masked_attn_asym(ctx: Context, feat: Features, Q, K, V, softmax=False, want_den=False):
    """Alg. 2 (asymmetric features: the mask estimate is Phi).  Q, K [G,N,m], V [G,N,d] CUDA tensors."""
    G, N, m = Q.shape
    d = V.shape[2]
    out = torch.empty_like(V)
    den = torch.empty((G, N), dtype=torch.float32, device=V.device) if want_den else None
    B.grf_masked_attn_asym(ctx.handle, feat.handle, G, N, m, d, B.dtype_code(Q),
                           B.GRF_KERNEL_SOFTMAX if softmax else B.GRF_KERNEL_LINEAR, Q, K, V, out, den)
    return (out, den) if want_den else out


def masked_attn_mhat(ctx: Context, feat: Features, phiQ, phiK, V, want_den=False):
    """Eqs. 1-2 over the materialised mask (call B.grf_features_materialise first).  bf16, d = 64."""
    G, N, m = phiQ.shape
    d = V.shape[2]
    out = torch.empty_like(V)
    den = torch.empty((G, N), dtype=torch.float32, device=V.device) if want_den else None
    B.grf_masked_attn_mhat(ctx.handle, feat.handle, G, N, m, d, B.dtype_code(phiQ), phiQ, phiK, V, out, den)
    return (out, den) if want_den else out
