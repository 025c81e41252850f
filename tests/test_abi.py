"""The C-ABI library loads without a GPU and exports every function include/grf.h declares."""
import ctypes
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "grf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(grf_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    from paper_2410_03462_b200 import binding
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(binding.lib, n), f"{n} is declared in grf.h but not exported by libgrf.so"
        assert n in binding.EXPORTED, f"{n} has no ctypes signature"
        assert callable(getattr(binding, n)), f"{n} has no Python wrapper of the same name"
    assert sorted(binding.EXPORTED) == names


def test_host_only_entry_points():
    from paper_2410_03462_b200 import binding as B
    f = B.grf_deconvolve([4.0, 4.0, 1.0])
    assert np.allclose(np.convolve(f, f)[:3], [4.0, 4.0, 1.0])
    try:
        B.grf_deconvolve([0.0, 1.0])
        raise AssertionError("alpha_0 = 0 must be rejected")
    except B.GrfError as e:
        assert e.code == B.GRF_ERR_INVALID
    assert B.grf_strerror(0) == "ok" and "workspace" in B.grf_strerror(B.GRF_ERR_WORKSPACE)
    one = B.grf_attn_workspace_bytes(1, 100, 32, 64, B.GRF_DTYPE_BF16)
    assert one >= 100 * 32 * 64 * 2 + 100 * 32 * 4 and one % 256 == 0
    assert B.grf_attn_workspace_bytes(7, 100, 32, 64, B.GRF_DTYPE_BF16) == 7 * one
    assert B.grf_attn_workspace_bytes(1, 100, 12, 64, B.GRF_DTYPE_BF16) == 0
    assert B.grf_attn_workspace_bytes(1, 100, 32, 64, 5) == 0


def test_no_cpu_fallback_without_a_device():
    """On a machine without a GPU the product path reports an error instead of computing elsewhere."""
    import torch
    if torch.cuda.is_available():
        return
    from paper_2410_03462_b200 import binding as B
    try:
        B.grf_ctx_create(0)
        raise AssertionError("context creation must fail without a CUDA device")
    except B.GrfError as e:
        assert e.code == B.GRF_ERR_CUDA


def test_product_code_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2410_03462_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in src, f"{fn} mentions the oracle"
    src = open(os.path.join(ROOT, "oracle", "__init__.py")).read() + open(os.path.join(ROOT, "oracle", "grf_oracle.c")).read()
    assert "paper_2410_03462_b200" not in src and "libgrf" not in src
