"""CPU oracle for GRF-masked linear attention — TEST INFRASTRUCTURE ONLY.

Plain, slow, obviously-correct code written from the paper; shares nothing with the CUDA
library.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import it.

Two layers:
  * `grf_oracle.c` (compiled on first use with gcc) — the sampler in the fp32/integer
    arithmetic the method's sampler is specified in, feature assembly (Eq. 10) and the fp64
    S/z-route attention (Eq. 12).
  * numpy functions below — definitions written out densely: the deconvolution of Remark 3.1,
    the power-series mask of Eq. 4 and the O(N^2) masked attention of Eqs. 1-2.

Pins (tests/test_oracle_*.py): Philox known answers; closed-form f for alpha_k = 2^-k;
(I - W/2)^-1; deterministic walks on a perfect matching; expected deposits per walk;
the L1 bound of Thm 3.2's proof; unbiasedness of Phi Psi^T; Lemma 3.3; brute force vs
S/z route; identity and all-ones features reducing to plain V / unmasked linear attention; the exp similarity
with an all-ones mask against scipy's softmax; Alg. 2's loop over walks against the dense definition with Mhat = Phi.
The order of equal columns inside a transposed row and the (walk, t) summation order are
fixed by this oracle's specification, not by the paper: parity unpinned by the paper for
those two orderings (they change no value beyond fp32 rounding order).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "grf_oracle.c")
_SO = os.path.join(_HERE, "_grf_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile grf_oracle.c with gcc (no fused multiply-add contraction, no fast-math)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_walks.restype = ctypes.c_int64
        _lib.oracle_features.restype = ctypes.c_int64
        _lib.oracle_attn_sparse.restype = ctypes.c_int
        _lib.oracle_philox4x32_10.restype = None
        _lib.oracle_transpose.restype = None
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


# ----------------------------------------------------------------------------- Philox

def philox4x32_10(ctr, key) -> np.ndarray:
    """One block of Philox4x32-10 (Salmon et al., SC'11)."""
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


# ----------------------------------------------------------------------------- Remark 3.1

def deconvolve(alpha) -> np.ndarray:
    """f with sum_{p<=k} f_p f_{k-p} = alpha_k (Remark 3.1), fp64; needs alpha_0 > 0."""
    alpha = np.asarray(alpha, dtype=np.float64)
    if alpha[0] <= 0:
        raise ValueError("alpha_0 must be positive")
    f = np.zeros_like(alpha)
    f[0] = np.sqrt(alpha[0])
    for k in range(1, len(alpha)):
        inner = 0.0
        for p in range(1, k):
            inner += f[p] * f[k - p]
        f[k] = (alpha[k] - inner) / (2.0 * f[0])
    return f


def power_series(W: np.ndarray, coeff) -> np.ndarray:
    """sum_k coeff_k W^k, dense fp64 (Eq. 4 with coeff = alpha; Remark 3.1 with coeff = f)."""
    W = np.asarray(W, dtype=np.float64)
    out = np.zeros_like(W)
    P = np.eye(W.shape[0])
    for c in np.asarray(coeff, dtype=np.float64):
        out += c * P
        P = P @ W
    return out


# ----------------------------------------------------------------------------- walks and features

@dataclass
class CSR:
    rowptr: np.ndarray  # int32 [rows+1]
    col: np.ndarray     # int32 [nnz]
    val: np.ndarray     # float32 [nnz]
    val64: np.ndarray | None  # fp64 shadow of val (error accounting), or None
    shape: tuple

    @property
    def nnz(self) -> int:
        return int(self.col.shape[0])

    def dense(self) -> np.ndarray:
        out = np.zeros(self.shape, dtype=np.float64)
        rows = np.repeat(np.arange(self.shape[0]), np.diff(self.rowptr))
        np.add.at(out, (rows, self.col), self.val.astype(np.float64))
        return out


def walks(rowptr, col, w, seed: int, n_walks: int, p_halt: float, max_len: int):
    """Trajectories [2,N,n,L+1] (int32, -1 after the end) and prefix loads (fp32) of both ensembles."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    col = np.ascontiguousarray(col, dtype=np.int32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    N = rowptr.shape[0] - 1
    traj = np.empty((2, N, n_walks, max_len + 1), dtype=np.int32)
    load = np.empty((2, N, n_walks, max_len + 1), dtype=np.float32)
    _load().oracle_walks(ctypes.c_int32(N), _p(rowptr), _p(col), _p(w), ctypes.c_uint64(seed),
                         ctypes.c_int32(n_walks), ctypes.c_float(p_halt), ctypes.c_int32(max_len),
                         _p(traj), _p(load))
    return traj, load


def features_from_walks(traj, load, e: int, f, keep_zero: bool = False) -> CSR:
    """Eq. 10 for ensemble e with modulation f (fp32 [L+1]).  Called again on the same walks with another f it is
    the re-modulation of Alg. 1's learnable (f_i) without re-walking.  keep_zero=True keeps the entries of prefixes
    whose coefficient is exactly 0 (as zeros), which makes the index structure independent of f."""
    _, N, n, Lp1 = traj.shape
    f = np.ascontiguousarray(f, dtype=np.float32)
    assert f.shape[0] == Lp1
    cap = N * n * Lp1
    rowptr = np.empty(N + 1, dtype=np.int32)
    col = np.empty(cap, dtype=np.int32)
    val = np.empty(cap, dtype=np.float32)
    val64 = np.empty(cap, dtype=np.float64)
    nnz = _load().oracle_features(ctypes.c_int32(N), ctypes.c_int32(n), ctypes.c_int32(Lp1 - 1),
                                  ctypes.c_int32(e), _p(traj), _p(load), _p(f),
                                  _p(rowptr), _p(col), _p(val), _p(val64), ctypes.c_int32(int(keep_zero)))
    if nnz < 0:
        raise MemoryError
    return CSR(rowptr, col[:nnz].copy(), val[:nnz].copy(), val64[:nnz].copy(), (N, N))


def transpose(a: CSR) -> CSR:
    rows, cols = a.shape
    t_rowptr = np.empty(cols + 1, dtype=np.int32)
    t_col = np.empty(a.nnz, dtype=np.int32)
    t_val = np.empty(a.nnz, dtype=np.float32)
    _load().oracle_transpose(ctypes.c_int32(rows), ctypes.c_int32(cols), _p(a.rowptr), _p(a.col), _p(a.val),
                             _p(t_rowptr), _p(t_col), _p(t_val))
    return CSR(t_rowptr, t_col, t_val, None, (cols, rows))


def sample(rowptr, col, w, seed, n_walks, p_halt, max_len, f_phi, f_psi=None, keep_zero: bool = False):
    """Alg. 1 steps 1-2 for two independent ensembles: returns (Phi, Psi, Psi^T, traj, load)."""
    traj, load = walks(rowptr, col, w, seed, n_walks, p_halt, max_len)
    if f_psi is None:
        f_psi = f_phi
    Phi = features_from_walks(traj, load, 0, f_phi, keep_zero)
    Psi = features_from_walks(traj, load, 1, f_psi, keep_zero)
    return Phi, Psi, transpose(Psi), traj, load


# ----------------------------------------------------------------------------- FLOP counts (Sec. 4, "Time complexity")

def flops_masked_linear(Phi: CSR, PsiT: CSR, m: int, d: int) -> int:
    """Floating-point operations of GRF-masked linear attention evaluated as Eq. 12, counted term by term for one
    problem: every non-zero Psi_jl costs one product with each of the m components of phi(k_j) and then one
    multiply-add into each of the d+1 columns of [S_l | z_l]; every non-zero Phi_il likewise against phi(q_i) and
    [S_l | z_l]; a multiply-add counts as 2; the N*d final divisions are added."""
    total = 0
    for l in range(PsiT.shape[0]):
        for _ in range(PsiT.rowptr[l], PsiT.rowptr[l + 1]):
            total += m + 2 * m * (d + 1)
    for i in range(Phi.shape[0]):
        for _ in range(Phi.rowptr[i], Phi.rowptr[i + 1]):
            total += m + 2 * m * (d + 1)
    return total + Phi.shape[0] * d


def flops_unmasked_linear(N: int, m: int, d: int) -> int:
    """Eq. 3 evaluated right to left: phi(K)^T [V | 1] (2 N m (d+1)), then phi(Q) times it (2 N m (d+1)), N d divisions."""
    return 4 * N * m * (d + 1) + N * d


def flops_softmax(N: int, m: int, d: int) -> int:
    """Unmasked softmax attention with query/key width m: scores 2 N^2 m, exponentials N^2, row sums N^2,
    weighted values 2 N^2 d, N d divisions."""
    return N * N * (2 * m + 2 + 2 * d) + N * d


# ----------------------------------------------------------------------------- attention

def attn_sparse(phiQ, phiK, V, Phi: CSR, PsiT: CSR, with_abs: bool = True):
    """Eq. 12 through S_l, z_l in fp64.  Inputs fp32 arrays [G,N,m]/[G,N,d] (exact storage values).
    Returns dict(num, den, out, num_abs, den_abs)."""
    phiQ = np.ascontiguousarray(phiQ, dtype=np.float32)
    phiK = np.ascontiguousarray(phiK, dtype=np.float32)
    V = np.ascontiguousarray(V, dtype=np.float32)
    G, N, m = phiQ.shape
    d = V.shape[2]
    R = Phi.shape[1]
    assert PsiT.shape == (R, N) and Phi.shape[0] == N
    num = np.empty((G, N, d)); den = np.empty((G, N))
    num_abs = np.empty((G, N, d)) if with_abs else None
    den_abs = np.empty((G, N)) if with_abs else None
    rc = _load().oracle_attn_sparse(ctypes.c_int32(G), ctypes.c_int32(N), ctypes.c_int32(R), ctypes.c_int32(m),
                                    ctypes.c_int32(d), _p(phiQ), _p(phiK), _p(V),
                                    _p(Phi.rowptr), _p(Phi.col), _p(Phi.val),
                                    _p(PsiT.rowptr), _p(PsiT.col), _p(PsiT.val),
                                    _p(num), _p(den),
                                    _p(num_abs) if with_abs else None, _p(den_abs) if with_abs else None)
    if rc != 0:
        raise MemoryError
    with np.errstate(divide="ignore", invalid="ignore"):
        out = np.where(den[..., None] != 0.0, num / den[..., None], 0.0)
    return dict(num=num, den=den, out=out, num_abs=num_abs, den_abs=den_abs)


def attn_bruteforce(phiQ, phiK, V, Mhat: np.ndarray, rows=None, kernel: str = "linear"):
    """Eqs. 1-2: A = S * Mhat, out = D^-1 A V, in fp64, with S = phiQ phiK^T (Eq. 3, kernel="linear") or
    S = exp(Q K^T) (softmax attention, kernel="exp").  `Mhat` is a dense N x N mask (e.g. Phi Psi^T, or Phi
    itself for asymmetric features).  `rows` optionally restricts the queries."""
    Q = np.asarray(phiQ, dtype=np.float64)
    K = np.asarray(phiK, dtype=np.float64)
    Vd = np.asarray(V, dtype=np.float64)
    G, N, _ = Q.shape
    rows = np.arange(N) if rows is None else np.asarray(rows)
    Mr = np.asarray(Mhat[rows], dtype=np.float64)      # only the requested rows of the mask are touched
    num = np.empty((G, len(rows), Vd.shape[2])); den = np.empty((G, len(rows)))
    num_abs = np.empty_like(num); den_abs = np.empty_like(den)
    for g in range(G):
        S = Q[g][rows] @ K[g].T
        A = (np.exp(S) if kernel == "exp" else S) * Mr
        num[g] = A @ Vd[g]
        den[g] = A.sum(axis=1)
        num_abs[g] = np.abs(A) @ np.abs(Vd[g])      # sums of the absolute values of the terms
        den_abs[g] = np.abs(A).sum(axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        out = np.where(den[..., None] != 0.0, num / den[..., None], 0.0)
    return dict(num=num, den=den, out=out, num_abs=num_abs, den_abs=den_abs)


def mask_rows(Phi: CSR, Psi: CSR, rows) -> np.ndarray:
    """Dense rows of Mhat = Phi Psi^T for the given query rows (Mhat_ij = sum_l Phi_il Psi_jl)."""
    PsiT = transpose(Psi)
    N = Psi.shape[0]
    out = np.zeros((len(rows), N))
    for r, i in enumerate(rows):
        for p in range(Phi.rowptr[i], Phi.rowptr[i + 1]):
            l = Phi.col[p]
            s, e = PsiT.rowptr[l], PsiT.rowptr[l + 1]
            np.add.at(out[r], PsiT.col[s:e], float(Phi.val[p]) * PsiT.val[s:e].astype(np.float64))
    return out


def materialise(Phi: CSR, Psi: CSR) -> CSR:
    """The mask estimate itself, Mhat = Phi Psi^T (Sec. 3.3: Mhat_ij = phi_hat(v_i)^T phi_hat(v_j)), as a sparse
    matrix: row i is sum_l Phi_il * (row l of Psi^T), accumulated in fp64 with l ascending; an entry exists iff
    some l has Phi_il and Psi_jl both stored (even if the products cancel).  `val` holds the fp32 rounding."""
    PsiT = transpose(Psi)
    N, Nk = Phi.shape[0], Psi.shape[0]
    rowptr = np.zeros(N + 1, dtype=np.int64)
    cols, vals = [], []
    acc = np.zeros(Nk)
    hit = np.zeros(Nk, dtype=bool)
    for i in range(N):
        touched = []
        for p in range(Phi.rowptr[i], Phi.rowptr[i + 1]):
            l = Phi.col[p]
            s, e = PsiT.rowptr[l], PsiT.rowptr[l + 1]
            js = PsiT.col[s:e]
            acc[js] += float(Phi.val[p]) * PsiT.val[s:e].astype(np.float64)   # the j of one row l are distinct
            hit[js] = True
            touched.append(js)
        if touched:
            js = np.unique(np.concatenate(touched))
            cols.append(js.astype(np.int32)); vals.append(acc[js].copy())
            acc[js] = 0.0; hit[js] = False
            rowptr[i + 1] = rowptr[i] + len(js)
        else:
            rowptr[i + 1] = rowptr[i]
    col = np.concatenate(cols) if cols else np.zeros(0, np.int32)
    val64 = np.concatenate(vals) if vals else np.zeros(0)
    return CSR(rowptr.astype(np.int32), col, val64.astype(np.float32), val64, (N, Nk))


def attn_asym_walks(Q, K, V, traj, load, f, kernel: str = "linear"):
    """Alg. 2 as printed (asymmetric features), in fp64, for ensemble 0 of `traj`/`load`: for every node i, every
    walk out of i and every step t of it, the visited node j contributes A_ij * f_t * load_t to the output
    feature (times v_j) and to the normalisation; the result is the quotient (the 1/n cancels)."""
    Qd = np.asarray(Q, dtype=np.float64); Kd = np.asarray(K, dtype=np.float64); Vd = np.asarray(V, dtype=np.float64)
    G, N, _ = Qd.shape
    _, _, n, Lp1 = traj.shape
    out = np.zeros((G, N, Vd.shape[2]))
    for g in range(G):
        for i in range(N):
            feat = np.zeros(Vd.shape[2]); norm = 0.0
            for k in range(n):
                for t in range(Lp1):
                    j = traj[0, i, k, t]
                    if j < 0:
                        break
                    s = float(Qd[g, i] @ Kd[g, j])
                    a = np.exp(s) if kernel == "exp" else s
                    wgt = a * float(f[t]) * float(load[0, i, k, t])
                    feat += wgt * Vd[g, j]; norm += wgt
            out[g, i] = feat / norm if norm != 0.0 else 0.0
    return out
