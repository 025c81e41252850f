"""Shared test helpers: oracle-side preparation of a workload and the comparison rules.

Tolerance rule for attention outputs (stated by the workloads' accuracy target: 1e-5 for fp32, 2e-2 for
bf16 storage, "relative"): with out = num/den, num and den sums of signed terms, an implementation whose
sums are each accurate to tol relative to the sum of the ABSOLUTE values of its terms satisfies
    |out' - out| <= tol * (num_abs + |out| * den_abs) / |den|
to first order.  For same-sign terms this is the plain relative error of den and the error of num on the
scale of its terms.  Rows whose denominator cancels almost completely (|den| < 1e-3 den_abs) are excluded
from the out comparison and checked through den alone.  num_abs and den_abs come from the oracle; they are pinned
against an independent dense computation in tests/test_oracle_pins.py (test_tolerance_scale_*)."""
from __future__ import annotations

import numpy as np

import oracle
from workloads import tensors

TOL = {"fp32": 1e-5, "bf16": 2e-2}


def oracle_features(w, g, seed, f_phi=None, f_psi=None):
    if f_phi is None:
        f_phi = oracle.deconvolve(w.alpha).astype(np.float32)
    return oracle.sample(g.rowptr, g.col, g.w, seed, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)


def assert_csr_equal(got, want: oracle.CSR, what: str, val_rtol=1e-5):
    rp, c, v = got
    assert np.array_equal(rp, want.rowptr), f"{what}: row pointers differ"
    assert np.array_equal(c, want.col), f"{what}: column indices differ"
    scale = np.maximum(np.abs(want.val), 1e-30)
    assert (np.abs(v - want.val) <= val_rtol * scale).all(), f"{what}: values differ"


def assert_attn_close(out_gpu: np.ndarray, ref: dict, tol: float, den_gpu: np.ndarray | None = None, what="",
                      min_ok: float = 0.9, same_sign: bool = False):
    """Compares outputs (and denominators) with an oracle result dict under the rule above.

    Rows without any feature (den_abs == 0) must come out as exact zeros and do not count as ill-conditioned.
    `same_sign=True` states that every term of every sum has one sign (non-negative features and phi(Q), phi(K)):
    then no row may be excluded, the denominators are compared by plain relative error and the outputs on the
    scale of the numerator's terms.  Returns the fraction of non-empty rows excluded as ill-conditioned."""
    out_gpu = np.asarray(out_gpu, dtype=np.float64)
    den, den_abs, num_abs, out = ref["den"], ref["den_abs"], ref["num_abs"], ref["out"]
    empty = den_abs == 0
    ok_rows = (np.abs(den) >= 1e-3 * den_abs) & ~empty
    nonempty = max(int((~empty).sum()), 1)
    excluded = 1.0 - ok_rows.sum() / nonempty
    if same_sign:
        assert np.allclose(den_abs, np.abs(den), rtol=1e-12, atol=0), f"{what}: terms are not of one sign"
        assert excluded == 0.0, f"{what}: rows excluded although all terms share a sign"
    assert 1.0 - excluded > min_ok, f"{what}: {excluded:.1%} of the rows are ill-conditioned"
    bound = tol * (num_abs + np.abs(out) * den_abs[..., None]) / np.maximum(np.abs(den), 1e-300)[..., None]
    err = np.abs(out_gpu - out)
    bad = (err > bound + 1e-30) & ok_rows[..., None]
    assert not bad.any(), f"{what}: {bad.sum()} outputs beyond tolerance, worst ratio {np.max(err[ok_rows] / (bound[ok_rows] + 1e-300)):.3g}"
    if den_gpu is not None:
        derr = np.abs(np.asarray(den_gpu, dtype=np.float64) - den)
        assert (derr <= tol * den_abs + 1e-30).all(), f"{what}: denominators beyond tolerance"
        if same_sign:
            assert (derr <= tol * np.abs(den) * (1 + 1e-12) + 1e-30).all(), f"{what}: denominators beyond plain relative tolerance"
    # rows with no features at all: Eq. 12 with an empty sum, out = 0 exactly
    if empty.any():
        assert (out_gpu[empty] == 0).all(), f"{what}: an empty feature row did not give zeros"
        if den_gpu is not None:
            assert (np.asarray(den_gpu)[empty] == 0).all(), f"{what}: an empty feature row has a non-zero denominator"
    return excluded


def qkv_for(w, N, G=None, seed=None):
    from workloads import configs
    return tensors.qkv(G or w.G, N, w.m, w.d, w.dtype, configs.QKV_SEED if seed is None else seed)
