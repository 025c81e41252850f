"""Parity at the benchmark's full size and launch configuration (N = 32768 point cloud, 8 heads, m = 32,
d = 64, bf16): the sampler's output bit for bit against the oracle, and the attention on sampled query rows
against the O(N) brute force of Eqs. 1-2 restricted to those rows."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers
from workloads import configs, tensors

pytestmark = pytest.mark.gpu


def test_bench_workload_sampler_and_sampled_attention_rows():
    from paper_2410_03462_b200 import api, binding as B
    w = configs.point_cloud_32768()
    g = w.graph()
    ctx = api.Context(0)
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f)
    for which, want in ((0, Phi), (1, Psi), (2, PsiT)):
        rp, c, v = feat.to_host(which)
        assert np.array_equal(rp, want.rowptr) and np.array_equal(c, want.col)
        assert np.array_equal(v.view(np.uint32), want.val.view(np.uint32))

    q, k, v = tensors.qkv(w.G, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 127, 128, g.N - 1], rng.integers(0, g.N, 260)]))
    assert len(rows) >= 256
    Mrows = oracle.mask_rows(Phi, Psi, rows)
    ref = oracle.attn_bruteforce(tensors.widen(q), tensors.widen(k), tensors.widen(v), Mrows_full(Mrows, rows, g.N), rows=rows)
    for tensor_cores in (True, False):
        B.grf_ctx_use_tensor_cores(ctx.handle, tensor_cores)
        out, den = api.masked_linear_attn(ctx, feat, qd, kd, vd, want_den=True)
        B.grf_ctx_check(ctx.handle)
        out_rows = out[:, rows].float().cpu().numpy()
        den_rows = den[:, rows].cpu().numpy()
        helpers.assert_attn_close(out_rows, ref, helpers.TOL["bf16"], den_rows, f"full size tensor_cores={tensor_cores}",
                                  same_sign=True)
        # properties that hold at any size: finite outputs, positive denominators (all terms are >= 0 here)
        assert torch.isfinite(out.float()).all()
        assert (den > 0).all()
    B.grf_ctx_use_tensor_cores(ctx.handle, True)
    # run-to-run determinism of the whole path at full size
    out2 = api.masked_linear_attn(ctx, feat, qd, kd, vd)
    out3 = api.masked_linear_attn(ctx, feat, qd, kd, vd)
    assert torch.equal(out2, out3)
    feat.free()
    ctx.close()


def test_bench_workload_asymmetric_route_sampled_rows():
    """Alg. 2 at the bench size (f_psi = delta_0, so the mask estimate is Phi): sampled query rows of both
    similarities against the brute force of Eqs. 1-2 on the dense rows of Phi."""
    from paper_2410_03462_b200 import api, binding as B
    w = configs.point_cloud_32768()
    g = w.graph()
    ctx = api.Context(0)
    f_phi = w.alpha.astype(np.float32)
    f_psi = np.zeros(w.max_len + 1, np.float32); f_psi[0] = 1.0
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f_phi, f_psi)
    assert Psi.nnz == g.N
    rng = np.random.default_rng(6)
    rows = np.unique(np.concatenate([[0, 7, 8, g.N - 1], rng.integers(0, g.N, 60)]))
    Mrows = np.zeros((len(rows), g.N))
    for r, i in enumerate(rows):
        s, e = Phi.rowptr[i], Phi.rowptr[i + 1]
        Mrows[r, Phi.col[s:e]] = Phi.val[s:e]
    q, k, v = tensors.qkv(w.G, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    for softmax in (False, True):
        qq, kk = (q, k) if not softmax else ((q.float() * 0.25).to(q.dtype), (k.float() * 0.25).to(k.dtype))
        ref = oracle.attn_bruteforce(tensors.widen(qq), tensors.widen(kk), tensors.widen(v), Mrows_full(Mrows, rows, g.N),
                                     rows=rows, kernel="exp" if softmax else "linear")
        out = api.masked_attn_asym(ctx, feat, qq.cuda(), kk.cuda(), v.cuda(), softmax=softmax)
        B.grf_ctx_check(ctx.handle)
        helpers.assert_attn_close(out[:, rows].float().cpu().numpy(), ref, helpers.TOL["bf16"], None,
                                  f"full size asymmetric softmax={softmax}")
        assert torch.isfinite(out.float()).all()
    feat.free()
    ctx.close()


def test_bench_workload_materialised_mask_route_sampled_rows():
    """Eqs. 1-2 over the materialised mask at the bench size and launch configuration: sampled rows of the stored mask
    against the oracle's rows of Phi Psi^T, and sampled query rows of the attention against the brute force."""
    from paper_2410_03462_b200 import api, binding as B
    w = configs.point_cloud_32768()
    g = w.graph()
    ctx = api.Context(0)
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f)
    B.grf_features_materialise(ctx.handle, feat.handle)
    B.grf_ctx_check(ctx.handle)
    rng = np.random.default_rng(8)
    rows = np.unique(np.concatenate([[0, 127, 128, g.N - 1], rng.integers(0, g.N, 260)]))
    assert len(rows) >= 256
    Mrows = oracle.mask_rows(Phi, Psi, rows)
    r_dev = torch.tensor(rows, dtype=torch.int32, device="cuda")
    got = torch.empty((len(rows), g.N), dtype=torch.float32, device="cuda")
    B.grf_mask_rows(ctx.handle, feat.handle, len(rows), r_dev, got)
    torch.cuda.synchronize()
    got = got.cpu().numpy().astype(np.float64)
    # one bf16 rounding of an fp32 sum of non-negative terms; values below the bf16 normal range may flush to zero
    assert (np.abs(got - Mrows) <= 2.0 ** -8 * np.abs(Mrows) + 1e-37).all()
    assert ((got != 0) <= (Mrows != 0)).all()
    q, k, v = tensors.qkv(w.G, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ref = oracle.attn_bruteforce(tensors.widen(q), tensors.widen(k), tensors.widen(v), Mrows_full(Mrows, rows, g.N), rows=rows)
    out, den = api.masked_attn_mhat(ctx, feat, qd, kd, vd, want_den=True)
    B.grf_ctx_check(ctx.handle)
    helpers.assert_attn_close(out[:, rows].float().cpu().numpy(), ref, helpers.TOL["bf16"], den[:, rows].cpu().numpy(),
                              "full size, materialised mask", same_sign=True)
    assert torch.isfinite(out.float()).all() and (den > 0).all()
    out2 = api.masked_attn_mhat(ctx, feat, qd, kd, vd)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    # and against the route through the per-node states on the same features (two roundings apart)
    out_sz = api.masked_linear_attn(ctx, feat, qd, kd, vd)
    torch.cuda.synchronize()
    a, b = out.float(), out_sz.float()
    assert ((a - b).abs() <= 4e-2 * (a.abs() + b.abs()) / 2 + 4e-2 * ref["num_abs"].max() / ref["den"].min()).all()
    feat.free()
    ctx.close()


def Mrows_full(Mrows, rows, N):
    """attn_bruteforce indexes the mask by absolute row: place the sampled rows into an N x N frame lazily."""
    class _Rows:
        def __init__(self):
            self.pos = {int(r): i for i, r in enumerate(rows)}
        def __getitem__(self, idx):
            return np.stack([Mrows[self.pos[int(r)]] for r in np.atleast_1d(idx)])
        def __array__(self, dtype=None, copy=None):
            raise TypeError("dense N x N mask is never formed")
    return _Rows()
