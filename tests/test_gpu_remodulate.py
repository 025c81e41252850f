"""GPU parity of re-modulation without re-walking (Alg. 1: learnable (f_i) on frozen walks) and of the operation
counts of Sec. 4, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers
from workloads import configs, graphs, tensors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2410_03462_b200 import api, binding
    ctx = api.Context(0)
    yield api, binding, ctx
    binding.grf_ctx_keep_walks(ctx.handle, False)
    ctx.close()


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def _assert_same_matrix(got, want: oracle.CSR, what):
    rp, c, v = got
    assert np.array_equal(rp, want.rowptr) and np.array_equal(c, want.col), f"{what}: structure differs"
    # bit for bit, except that a zero may carry either sign
    same = (_bits(v) == _bits(want.val)) | ((v == 0) & (want.val == 0))
    assert same.all(), f"{what}: {np.count_nonzero(~same)} values differ"


CASES = {
    "tiny": lambda: configs.tiny(),
    "vit": lambda: configs.vit_grid(),                 # mixed-sign coefficients
    "pc1024": lambda: configs.point_cloud_4096(1024),
    "reg2048": lambda: configs.sweep(11),
}


@pytest.mark.parametrize("name", list(CASES))
def test_kept_walks_and_remodulation_bit_exact(lib, name):
    api, B, ctx = lib
    w = CASES[name]()
    g = w.graph()
    dg = api.DeviceGraph(g)
    rng = np.random.default_rng(5)
    f0 = oracle.deconvolve(w.alpha).astype(np.float32)
    f0[min(3, w.max_len)] = 0.0                         # a zero coefficient: the kept structure must not notice
    traj, load = oracle.walks(g.rowptr, g.col, g.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len)
    B.grf_ctx_keep_walks(ctx.handle, True)
    feat = api.sample(ctx, dg, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f0)
    for e in (0, 1):
        _assert_same_matrix(feat.to_host(e), oracle.features_from_walks(traj, load, e, f0, keep_zero=True), f"kept {e}")
    # entries that plain sampling creates carry the same bits
    B.grf_ctx_keep_walks(ctx.handle, False)
    plain = api.sample(ctx, dg, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f0)
    prp, pc, pv = plain.to_host(0)
    krp, kc, kv = feat.to_host(0)
    for i in range(0, g.N, max(1, g.N // 64)):
        kept_row = dict(zip(kc[krp[i]:krp[i + 1]].tolist(), kv[krp[i]:krp[i + 1]]))
        for c, v in zip(pc[prp[i]:prp[i + 1]].tolist(), pv[prp[i]:prp[i + 1]]):
            assert _bits(kept_row[c]) == _bits(v) or (kept_row[c] == 0 and v == 0)
    plain.free()
    # new coefficients, two rounds, different for the two ensembles
    for rnd in range(2):
        f_phi = rng.standard_normal(w.max_len + 1).astype(np.float32)
        f_psi = rng.standard_normal(w.max_len + 1).astype(np.float32)
        if rnd == 1:
            f_psi[1] = 0.0
        B.grf_remodulate(ctx.handle, feat.handle, w.max_len, f_phi, f_psi)
        Phi = oracle.features_from_walks(traj, load, 0, f_phi, keep_zero=True)
        Psi = oracle.features_from_walks(traj, load, 1, f_psi, keep_zero=True)
        _assert_same_matrix(feat.to_host(0), Phi, "remodulated Phi")
        _assert_same_matrix(feat.to_host(1), Psi, "remodulated Psi")
        _assert_same_matrix(feat.to_host(2), oracle.transpose(Psi), "remodulated Psi^T")
    # the same coefficients by fresh walks with the same seed: identical object
    B.grf_ctx_keep_walks(ctx.handle, True)
    fresh = api.sample(ctx, dg, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
    B.grf_ctx_keep_walks(ctx.handle, False)
    for which in (0, 1, 2):
        a, b = feat.to_host(which), fresh.to_host(which)
        assert all(np.array_equal(x, y) for x, y in zip(a[:2], b[:2])) and np.array_equal(_bits(a[2]), _bits(b[2]))
    fresh.free()
    feat.free()


def test_attention_after_remodulation_matches_oracle(lib):
    """The attention (both gather kernels) must see the new values: the block plan's coefficient table is rebuilt."""
    api, B, ctx = lib
    w = configs.point_cloud_4096(1024)
    g = w.graph()
    f0 = oracle.deconvolve(w.alpha).astype(np.float32)
    B.grf_ctx_keep_walks(ctx.handle, True)
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f0)
    B.grf_ctx_keep_walks(ctx.handle, False)
    q, k, v = tensors.qkv(2, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    api.masked_linear_attn(ctx, feat, qd, kd, vd)            # builds the plan for the old values
    f1 = (f0 * np.linspace(1.0, 0.2, w.max_len + 1)).astype(np.float32)
    B.grf_remodulate(ctx.handle, feat.handle, w.max_len, f1, None)
    traj, load = oracle.walks(g.rowptr, g.col, g.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len)
    Phi = oracle.features_from_walks(traj, load, 0, f1, keep_zero=True)
    PsiT = oracle.transpose(oracle.features_from_walks(traj, load, 1, f1, keep_zero=True))
    ref = oracle.attn_sparse(tensors.widen(q), tensors.widen(k), tensors.widen(v), Phi, PsiT)
    for tensor_cores in (True, False):
        B.grf_ctx_use_tensor_cores(ctx.handle, tensor_cores)
        out, den = api.masked_linear_attn(ctx, feat, qd, kd, vd, want_den=True)
        B.grf_ctx_check(ctx.handle)
        helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL["bf16"], den.cpu().numpy(),
                                  f"after remodulation, tensor_cores={tensor_cores}", same_sign=True)
    B.grf_ctx_use_tensor_cores(ctx.handle, True)
    feat.free()


def test_mask_after_remodulation_rebuilds_values_only_and_matches_a_full_build(lib):
    """The materialised mask after new coefficients: its key lists and positions are kept (same walks, same
    structure), only the values are formed again; they must equal, bit for bit, those of a mask built from scratch
    on a fresh object with the same coefficients, and the oracle's rows of Phi Psi^T within the bf16 bound."""
    api, B, ctx = lib
    w = configs.point_cloud_4096(1000)                       # ragged last block
    g = w.graph()
    N = g.N
    dg = api.DeviceGraph(g)
    f0 = oracle.deconvolve(w.alpha).astype(np.float32)
    f1 = (f0 * np.linspace(1.0, -0.3, w.max_len + 1)).astype(np.float32)      # mixed signs
    f1[2] = 0.0
    B.grf_ctx_keep_walks(ctx.handle, True)
    feat = api.sample(ctx, dg, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f0)
    fresh = api.sample(ctx, dg, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f1)
    B.grf_ctx_keep_walks(ctx.handle, False)
    B.grf_features_materialise(ctx.handle, feat.handle)      # structure and values for f0
    stats0 = B.grf_mask_stats(feat.handle)
    launches0 = ctx.launches
    B.grf_features_materialise(ctx.handle, fresh.handle)
    full_build = ctx.launches - launches0
    B.grf_remodulate(ctx.handle, feat.handle, w.max_len, f1, None)
    with pytest.raises(B.GrfError):                           # the old values are not served
        B.grf_mask_stats(feat.handle)
    launches0 = ctx.launches
    B.grf_features_materialise(ctx.handle, feat.handle)
    assert ctx.launches - launches0 == 1 < full_build         # the values kernel alone
    assert B.grf_mask_stats(feat.handle) == stats0 == B.grf_mask_stats(fresh.handle)
    rows = torch.arange(N, dtype=torch.int32, device="cuda")
    a = torch.empty((N, N), dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    B.grf_mask_rows(ctx.handle, feat.handle, N, rows, a)
    B.grf_mask_rows(ctx.handle, fresh.handle, N, rows, b)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    traj, load = oracle.walks(g.rowptr, g.col, g.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len)
    Phi = oracle.features_from_walks(traj, load, 0, f1, keep_zero=True)
    Psi = oracle.features_from_walks(traj, load, 1, f1, keep_zero=True)
    sel = sorted(set([0, 1, N // 2, N - 1] + list(range(0, N, 29))))
    want = oracle.mask_rows(Phi, Psi, sel)
    got = a[sel].cpu().numpy().astype(np.float64)
    assert (np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-37).all()
    # and the attention over it
    q, k, v = tensors.qkv(2, N, w.m, 64, "bf16", configs.QKV_SEED)
    out1 = api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    out2 = api.masked_attn_mhat(ctx, fresh, q.cuda(), k.cuda(), v.cuda())
    torch.cuda.synchronize()
    B.grf_ctx_check(ctx.handle)
    assert torch.equal(out1, out2)
    # resampling drops the structure as well
    feat.handle = B.grf_sample(ctx.handle, N, dg.rowptr, dg.col, dg.w, configs.WALK_SEED + 1, w.n_walks, w.p_halt, w.max_len,
                               f1, None, feat.handle)
    launches0 = ctx.launches
    B.grf_features_materialise(ctx.handle, feat.handle)
    assert ctx.launches - launches0 > 1
    feat.free()
    fresh.free()


def test_remodulate_rejects_objects_without_deposits(lib):
    api, B, ctx = lib
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    B.grf_ctx_keep_walks(ctx.handle, False)
    feat = api.sample(ctx, api.DeviceGraph(g), 1, w.n_walks, w.p_halt, w.max_len, f)
    with pytest.raises(B.GrfError) as e:
        B.grf_remodulate(ctx.handle, feat.handle, w.max_len, f, None)
    assert e.value.code == B.GRF_ERR_INVALID
    B.grf_ctx_keep_walks(ctx.handle, True)
    api.sample(ctx, api.DeviceGraph(g), 1, w.n_walks, w.p_halt, w.max_len, f, features=feat)
    B.grf_ctx_keep_walks(ctx.handle, False)
    with pytest.raises(B.GrfError):
        B.grf_remodulate(ctx.handle, feat.handle, w.max_len - 1, f[:-1], None)     # another max_len than sampled
    B.grf_remodulate(ctx.handle, feat.handle, w.max_len, f, None)
    feat.free()


def test_flop_counts_match_oracle_and_grow_linearly(lib):
    """Sec. 4 "Time complexity": 1-D grids, n = 4, p_halt = 0.5, m = d = 8, mean over 10 seeds."""
    api, B, ctx = lib
    m = d = 8
    L = 8
    f = oracle.deconvolve(0.5 ** np.arange(L + 1)).astype(np.float32)
    means = {}
    for N in (256, 512, 1024):
        g = graphs.path_graph(N, 0.5)
        dg = api.DeviceGraph(g)
        counts = []
        for seed in range(10):
            feat = api.sample(ctx, dg, seed, 4, 0.5, L, f)
            masked, linear, softmax = B.grf_attn_flops(feat.handle, m, d)
            if seed < 2:
                Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, seed, 4, 0.5, L, f)
                assert masked == oracle.flops_masked_linear(Phi, PsiT, m, d)
            assert linear == oracle.flops_unmasked_linear(N, m, d) and softmax == oracle.flops_softmax(N, m, d)
            counts.append(masked)
            feat.free()
        means[N] = float(np.mean(counts))
    assert abs(means[512] / means[256] - 2) < 0.05 and abs(means[1024] / means[512] - 2) < 0.05
