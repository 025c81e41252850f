"""Thin ctypes binding of the C-ABI library: argument marshalling only.

Function names match include/grf.h.  Device pointers may be given as torch CUDA tensors (their
data_ptr() is passed) or as plain integers; host arrays as numpy arrays.  Every computing call goes to
the CUDA library; if the library cannot be loaded the import of this module fails."""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

GRF_OK = 0
GRF_ERR_INVALID, GRF_ERR_TOO_LARGE, GRF_ERR_WORKSPACE, GRF_ERR_CUDA, GRF_ERR_NOMEM, GRF_ERR_BADGRAPH = -1, -2, -3, -4, -5, -6
GRF_ERR_TIMEOUT = -7
GRF_DTYPE_F32, GRF_DTYPE_BF16 = 0, 1
GRF_KERNEL_LINEAR, GRF_KERNEL_SOFTMAX = 0, 1

_LIB_PATH = _build.LIB
if not os.path.exists(_LIB_PATH):
    _build.build()
lib = ctypes.CDLL(_LIB_PATH)

_vp, _i32, _i64, _u64, _f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_float
_sz, _int = ctypes.c_size_t, ctypes.c_int

_SIGNATURES = {
    "grf_ctx_create": (_int, [ctypes.POINTER(_vp), _int, _vp]),
    "grf_ctx_destroy": (_int, [_vp]),
    "grf_deconvolve": (_int, [_vp, _i32, _vp]),
    "grf_sample": (_int, [_vp, _i32, _vp, _vp, _vp, _u64, _i32, _f32, _i32, _vp, _vp, ctypes.POINTER(_vp)]),
    "grf_ctx_keep_walks": (_int, [_vp, _int]),
    "grf_remodulate": (_int, [_vp, _vp, _i32, _vp, _vp]),
    "grf_attn_flops": (_int, [_vp, _i32, _i32, ctypes.POINTER(_i64), ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "grf_debug_walks": (_int, [_vp, _i32, _vp, _vp, _vp, _u64, _i32, _f32, _i32, _vp, _vp]),
    "grf_features_from_csr": (_int, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.POINTER(_vp)]),
    "grf_features_view": (_int, [_vp, _int, ctypes.POINTER(_i32), ctypes.POINTER(_i32), ctypes.POINTER(_i64),
                                 ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp)]),
    "grf_features_copy": (_int, [_vp, _vp, _int, _vp, _vp, _vp]),
    "grf_features_free": (_int, [_vp]),
    "grf_csr_transpose": (_int, [_vp, _i32, _i32, _i64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "grf_csr_transpose_noalloc": (_int, [_int, _vp, _i32, _i32, _i64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "grf_attn_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32, _int]),
    "grf_masked_linear_attn": (_int, [_vp, _vp, _i32, _i32, _i32, _i32, _int, _vp, _vp, _vp, _vp, _vp, _vp, _sz]),
    "grf_masked_attn_asym": (_int, [_vp, _vp, _i32, _i32, _i32, _i32, _int, _int, _vp, _vp, _vp, _vp, _vp]),
    "grf_features_materialise": (_int, [_vp, _vp]),
    "grf_mask_stats": (_int, [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "grf_mask_rows": (_int, [_vp, _vp, _i32, _vp, _vp]),
    "grf_masked_attn_mhat": (_int, [_vp, _vp, _i32, _i32, _i32, _i32, _int, _vp, _vp, _vp, _vp, _vp]),
    "grf_step_host": (_int, [_vp, _i32, _vp, _vp, _vp, _u64, _i32, _f32, _i32, _vp, _vp,
                             _i32, _i32, _i32, _int, _vp, _vp, _vp, _vp]),
    "grf_plan_stats": (_int, [_vp, _vp, ctypes.POINTER(_i32), ctypes.POINTER(_i64)]),
    "grf_ctx_launch_count": (_i64, [_vp]),
    "grf_ctx_check": (_int, [_vp]),
    "grf_debug_wait_timeout": (_int, [_vp, _i64]),
    "grf_ctx_check_graphs": (_int, [_vp, _int]),
    "grf_ctx_prefer_mask_route": (_int, [_vp, _int]),
    "grf_ctx_use_tensor_cores": (_int, [_vp, _int]),
    "grf_ctx_enable_timing": (_int, [_vp, _int]),
    "grf_ctx_kernel_times": (_int, [_vp, _vp, _vp]),
    "grf_strerror": (ctypes.c_char_p, [_int]),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype, _fn.argtypes = _res, _args

EXPORTED = tuple(_SIGNATURES)


class GrfError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib.grf_strerror(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != GRF_OK:
        raise GrfError(code, where)


def _dev(x):
    """Device address of a torch CUDA tensor, or an int passed through; None -> NULL."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return x.data_ptr()


def _host(x, dtype):
    """Host address of a numpy array of the given dtype (kept alive by the caller); None -> NULL."""
    if x is None:
        return None, None
    a = np.ascontiguousarray(x, dtype=dtype)
    return a.ctypes.data, a


def dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return GRF_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return GRF_DTYPE_BF16
    raise ValueError(f"unsupported dtype {t.dtype}")


def grf_ctx_create(device: int = 0, stream: int | None = None) -> int:
    h = _vp()
    _check(lib.grf_ctx_create(ctypes.byref(h), device, stream), "grf_ctx_create")
    return h.value


def grf_ctx_destroy(ctx: int):
    _check(lib.grf_ctx_destroy(ctx), "grf_ctx_destroy")


def grf_plan_stats(ctx, features):
    """(blocks, node-list entries over all blocks) of the tensor-core gather's block plan."""
    b, e = _i32(), _i64()
    _check(lib.grf_plan_stats(ctx, features, ctypes.byref(b), ctypes.byref(e)), "grf_plan_stats")
    return b.value, e.value


def grf_ctx_launch_count(ctx: int) -> int:
    return int(lib.grf_ctx_launch_count(ctx))


def grf_ctx_check(ctx: int):
    _check(lib.grf_ctx_check(ctx), "grf_ctx_check")


def grf_debug_wait_timeout(ctx: int, limit_cycles: int):
    _check(lib.grf_debug_wait_timeout(ctx, limit_cycles), "grf_debug_wait_timeout")


def grf_ctx_prefer_mask_route(ctx: int, enable: bool):
    _check(lib.grf_ctx_prefer_mask_route(ctx, int(enable)), "grf_ctx_prefer_mask_route")


def grf_ctx_check_graphs(ctx: int, enable: bool):
    _check(lib.grf_ctx_check_graphs(ctx, int(enable)), "grf_ctx_check_graphs")


def grf_ctx_use_tensor_cores(ctx: int, enable: bool):
    _check(lib.grf_ctx_use_tensor_cores(ctx, int(enable)), "grf_ctx_use_tensor_cores")


KERNEL_CLASSES = ("walk_merge", "scan", "compact", "regroup", "build_states", "gather_contract", "row_denominators",
                  "block_plan", "mask_build", "mhat_attention")


def grf_ctx_enable_timing(ctx: int, enable: bool):
    _check(lib.grf_ctx_enable_timing(ctx, int(enable)), "grf_ctx_enable_timing")


def grf_ctx_kernel_times(ctx: int):
    """{class name: (milliseconds, timed launch groups)} since the previous read."""
    ms = np.zeros(len(KERNEL_CLASSES), dtype=np.float32)
    n = np.zeros(len(KERNEL_CLASSES), dtype=np.int64)
    _check(lib.grf_ctx_kernel_times(ctx, ms.ctypes.data, n.ctypes.data), "grf_ctx_kernel_times")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_CLASSES)}


def grf_deconvolve(alpha) -> np.ndarray:
    a = np.ascontiguousarray(alpha, dtype=np.float64)
    f = np.empty_like(a)
    _check(lib.grf_deconvolve(a.ctypes.data, a.shape[0], f.ctypes.data), "grf_deconvolve")
    return f


def grf_sample(ctx, N, rowptr, col, w, seed, n_walks, p_halt, max_len, f_phi, f_psi=None, features=None) -> int:
    """Returns the feature-object handle (a new one, or `features` refilled)."""
    p_phi, k1 = _host(f_phi, np.float32)
    p_psi, k2 = _host(f_psi, np.float32)
    if k1 is None or k1.shape[0] != max_len + 1 or (k2 is not None and k2.shape[0] != max_len + 1):
        raise ValueError("modulation arrays must hold max_len + 1 coefficients")
    h = _vp(features)
    _check(lib.grf_sample(ctx, N, _dev(rowptr), _dev(col), _dev(w), seed, n_walks, p_halt, max_len,
                          p_phi, p_psi, ctypes.byref(h)), "grf_sample")
    return h.value


def grf_ctx_keep_walks(ctx: int, enable: bool):
    _check(lib.grf_ctx_keep_walks(ctx, int(enable)), "grf_ctx_keep_walks")


def grf_remodulate(ctx, features, max_len, f_phi, f_psi=None):
    p_phi, k1 = _host(f_phi, np.float32)
    p_psi, k2 = _host(f_psi, np.float32)
    if k1 is None or k1.shape[0] != max_len + 1 or (k2 is not None and k2.shape[0] != max_len + 1):
        raise ValueError("modulation arrays must hold max_len + 1 coefficients")
    _check(lib.grf_remodulate(ctx, features, max_len, p_phi, p_psi), "grf_remodulate")


def grf_attn_flops(features, m, d):
    """(masked, unmasked_linear, softmax) operation counts of one problem."""
    a, b, c = _i64(), _i64(), _i64()
    _check(lib.grf_attn_flops(features, m, d, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "grf_attn_flops")
    return a.value, b.value, c.value


def grf_debug_walks(ctx, N, rowptr, col, w, seed, n_walks, p_halt, max_len, traj, load):
    _check(lib.grf_debug_walks(ctx, N, _dev(rowptr), _dev(col), _dev(w), seed, n_walks, p_halt, max_len,
                               _dev(traj), _dev(load)), "grf_debug_walks")


def grf_features_from_csr(ctx, N, R, phi_rowptr, phi_col, phi_val, psi_rowptr, psi_col, psi_val) -> int:
    h = _vp()
    _check(lib.grf_features_from_csr(ctx, N, R, _dev(phi_rowptr), _dev(phi_col), _dev(phi_val),
                                     _dev(psi_rowptr), _dev(psi_col), _dev(psi_val), ctypes.byref(h)),
           "grf_features_from_csr")
    return h.value


def grf_features_view(features: int, which: int):
    """(rows, cols, nnz, rowptr_ptr, col_ptr, val_ptr): borrowed device addresses."""
    rows, cols, nnz = _i32(), _i32(), _i64()
    rp, cp, vp = _vp(), _vp(), _vp()
    _check(lib.grf_features_view(features, which, ctypes.byref(rows), ctypes.byref(cols), ctypes.byref(nnz),
                                 ctypes.byref(rp), ctypes.byref(cp), ctypes.byref(vp)), "grf_features_view")
    return rows.value, cols.value, nnz.value, rp.value, cp.value, vp.value


def grf_features_copy(ctx, features, which, rowptr, col, val):
    _check(lib.grf_features_copy(ctx, features, which, _dev(rowptr), _dev(col), _dev(val)), "grf_features_copy")


def grf_features_free(features: int):
    _check(lib.grf_features_free(features), "grf_features_free")


def grf_csr_transpose(ctx, rows, cols, nnz, rowptr, col, val, t_rowptr, t_col, t_val):
    _check(lib.grf_csr_transpose(ctx, rows, cols, nnz, _dev(rowptr), _dev(col), _dev(val),
                                 _dev(t_rowptr), _dev(t_col), _dev(t_val)), "grf_csr_transpose")


def grf_csr_transpose_noalloc(device, stream, rows, cols, nnz, rowptr, col, val, t_rowptr, t_col, t_val):
    """Allocation-free variant of grf_csr_transpose (fixed in-library scratch; see grf.h for its limits)."""
    _check(lib.grf_csr_transpose_noalloc(device, stream, rows, cols, nnz, _dev(rowptr), _dev(col), _dev(val),
                                         _dev(t_rowptr), _dev(t_col), _dev(t_val)), "grf_csr_transpose_noalloc")


def grf_attn_workspace_bytes(G, R, m, d, dtype) -> int:
    return int(lib.grf_attn_workspace_bytes(G, R, m, d, dtype))


def grf_masked_linear_attn(ctx, features, G, N, m, d, dtype, phiQ, phiK, V, out, den_out, workspace,
                           workspace_bytes):
    _check(lib.grf_masked_linear_attn(ctx, features, G, N, m, d, dtype, _dev(phiQ), _dev(phiK), _dev(V),
                                      _dev(out), _dev(den_out), _dev(workspace), workspace_bytes),
           "grf_masked_linear_attn")


def grf_masked_attn_asym(ctx, features, G, N, m, d, dtype, kernel, Q, K, V, out, den_out):
    _check(lib.grf_masked_attn_asym(ctx, features, G, N, m, d, dtype, kernel, _dev(Q), _dev(K), _dev(V), _dev(out),
                                    _dev(den_out)), "grf_masked_attn_asym")


def grf_features_materialise(ctx, features):
    _check(lib.grf_features_materialise(ctx, features), "grf_features_materialise")


def grf_mask_stats(features):
    """(blocks, key entries over all blocks, device bytes)."""
    b, e, n = _i32(), _i64(), _i64()
    _check(lib.grf_mask_stats(features, ctypes.byref(b), ctypes.byref(e), ctypes.byref(n)), "grf_mask_stats")
    return b.value, e.value, n.value


def grf_mask_rows(ctx, features, n, rows, out):
    _check(lib.grf_mask_rows(ctx, features, n, _dev(rows), _dev(out)), "grf_mask_rows")


def grf_masked_attn_mhat(ctx, features, G, N, m, d, dtype, phiQ, phiK, V, out, den_out):
    _check(lib.grf_masked_attn_mhat(ctx, features, G, N, m, d, dtype, _dev(phiQ), _dev(phiK), _dev(V), _dev(out),
                                    _dev(den_out)), "grf_masked_attn_mhat")


def grf_step_host(ctx, N, rowptr, col, w, seed, n_walks, p_halt, max_len, f_phi, f_psi, G, m, d, dtype,
                  phiQ, phiK, V, out):
    """All array arguments are HOST addresses (ints) or numpy arrays / CPU torch tensors."""
    def haddr(x):
        if x is None or isinstance(x, int):
            return x
        if isinstance(x, np.ndarray):
            return x.ctypes.data
        return x.data_ptr()
    p_phi, k1 = _host(f_phi, np.float32)
    p_psi, k2 = _host(f_psi, np.float32)
    _check(lib.grf_step_host(ctx, N, haddr(rowptr), haddr(col), haddr(w), seed, n_walks, p_halt, max_len,
                             p_phi, p_psi, G, m, d, dtype, haddr(phiQ), haddr(phiK), haddr(V), haddr(out)),
           "grf_step_host")


def grf_strerror(code: int) -> str:
    return lib.grf_strerror(code).decode()
