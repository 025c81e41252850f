"""GPU parity of the route through the materialised mask (Eqs. 1-2 with Mhat = Phi Psi^T): the mask blocks against
the oracle's rows of Phi Psi^T, and the attention against the dense definition."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers
from workloads import configs, tensors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2410_03462_b200 import api, binding
    ctx = api.Context(0)
    yield api, binding, ctx
    ctx.close()


def _mask_rows(B, ctx, feat, rows, N):
    r = torch.tensor(rows, dtype=torch.int32, device="cuda")
    out = torch.empty((len(rows), N), dtype=torch.float32, device="cuda")
    B.grf_mask_rows(ctx.handle, feat.handle, len(rows), r, out)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


def _check_mask(got, want, what):
    """bf16 storage of an fp32 sum: half an ulp of bf16 (2^-9) relative, plus the fp32 rounding of the sum on the
    scale of its terms (covered by a small multiple), and underflow to zero below the bf16 normal range."""
    err = np.abs(got - want)
    bound = 2.0 ** -8 * np.abs(want) + 1e-37
    assert (err <= bound).all(), f"{what}: mask values differ, worst ratio {np.max(err / bound):.3g}"
    assert ((got != 0) <= (want != 0)).all(), f"{what}: an entry outside the support of Phi Psi^T is non-zero"


CASES = {
    "tiny64": (lambda: configs.tiny(), 1, None),
    "pc1000": (lambda: configs.point_cloud_4096(1000), 2, None),        # ragged last block
    "pc2048": (lambda: configs.point_cloud_4096(2048), 3, None),
    "vit": (lambda: configs.vit_grid(), 12, None),                      # mixed-sign coefficients, m = 64
    "reg1024": (lambda: configs.sweep(10), 2, None),                    # no locality: every block reaches every key
}


@pytest.mark.parametrize("name", list(CASES))
def test_mask_blocks_and_attention_match_oracle(lib, name):
    api, B, ctx = lib
    make, G, _ = CASES[name]
    w = make()
    g = w.graph()
    N = g.N
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f)
    B.grf_features_materialise(ctx.handle, feat.handle)
    blocks, entries, nbytes = B.grf_mask_stats(feat.handle)
    assert blocks == (N + 127) // 128 and entries % 64 == 0 and nbytes == entries * 260
    rows = sorted(set([0, 1, N // 2, N - 1] + list(range(0, N, max(1, N // 37)))))
    want = oracle.mask_rows(Phi, Psi, rows)
    _check_mask(_mask_rows(B, ctx, feat, rows, N), want, name)
    # attention against the dense definition with the oracle's own mask
    q, k, v = tensors.qkv(G, N, w.m, 64, "bf16", configs.QKV_SEED)
    M = oracle.mask_rows(Phi, Psi, list(range(N))) if N <= 2048 else None
    ref = oracle.attn_bruteforce(tensors.widen(q), tensors.widen(k), tensors.widen(v), M)
    out, den = api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda(), want_den=True)
    B.grf_ctx_check(ctx.handle)
    helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL["bf16"], den.cpu().numpy(), name,
                              same_sign=(name != "vit"))
    # and it is the same function as the route through the per-node states
    ref2 = oracle.attn_sparse(tensors.widen(q), tensors.widen(k), tensors.widen(v), Phi, PsiT)
    helpers.assert_attn_close(out.float().cpu().numpy(), ref2, helpers.TOL["bf16"], den.cpu().numpy(), name + " (S/z oracle)",
                              same_sign=(name != "vit"))
    # run-to-run identical, mask rebuilt
    B.grf_features_materialise(ctx.handle, feat.handle)
    out2 = api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    feat.free()


@pytest.mark.parametrize("m", [16, 32, 64])
def test_signed_rectangular_features_and_empty_rows(lib, m):
    """Phi, Psi are N x R with R != N, signed values, some empty rows of Phi (out = 0 exactly) and of Psi."""
    import scipy.sparse as sp
    api, B, ctx = lib
    rng = np.random.default_rng(m)
    N, R, G = 300, 517, 2

    def rand_csr(density, empty_rows):
        A = sp.random(N, R, density, random_state=int(rng.integers(1 << 30)), data_rvs=rng.standard_normal, format="csr")
        A = A.tolil()
        for r in empty_rows:
            A[r, :] = 0
        A = A.tocsr(); A.eliminate_zeros(); A.sort_indices()
        return oracle.CSR(A.indptr.astype(np.int32), A.indices.astype(np.int32), A.data.astype(np.float32), None, (N, R))

    Phi = rand_csr(0.03, [0, 5, 299])
    Psi = rand_csr(0.03, [7, 128])
    feat = api.features_from_csr(ctx, N, R, (Phi.rowptr, Phi.col, Phi.val), (Psi.rowptr, Psi.col, Psi.val))
    B.grf_features_materialise(ctx.handle, feat.handle)
    rows = list(range(0, N, 7)) + [299]
    _check_mask(_mask_rows(B, ctx, feat, rows, N), oracle.mask_rows(Phi, Psi, rows), f"m={m}")
    q, k, v = tensors.qkv(G, N, m, 64, "bf16", 77)
    k = (k.float() - 0.3).to(torch.bfloat16)          # signed key features as well
    M = oracle.mask_rows(Phi, Psi, list(range(N)))
    ref = oracle.attn_bruteforce(tensors.widen(q), tensors.widen(k), tensors.widen(v), M)
    out, den = api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda(), want_den=True)
    B.grf_ctx_check(ctx.handle)
    helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL["bf16"], den.cpu().numpy(), f"m={m}", min_ok=0.5)
    feat.free()


def test_mask_is_dropped_by_resampling_and_shapes_are_checked(lib):
    api, B, ctx = lib
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g), 3, w.n_walks, w.p_halt, w.max_len, f)
    q, k, v = tensors.qkv(1, g.N, 32, 64, "bf16", 1)
    with pytest.raises(B.GrfError):                       # no mask yet
        api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    with pytest.raises(B.GrfError):
        B.grf_mask_stats(feat.handle)
    B.grf_features_materialise(ctx.handle, feat.handle)
    api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    q8, k8, _ = tensors.qkv(1, g.N, 8, 64, "bf16", 1)
    with pytest.raises(B.GrfError) as e:                  # m = 8 is not covered by this route
        api.masked_attn_mhat(ctx, feat, q8.cuda(), k8.cuda(), v.cuda())
    assert e.value.code == B.GRF_ERR_INVALID
    api.sample(ctx, api.DeviceGraph(g), 4, w.n_walks, w.p_halt, w.max_len, f, features=feat)
    with pytest.raises(B.GrfError):                       # resampled: the old mask must not be used
        api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    B.grf_ctx_check(ctx.handle)
    feat.free()


def test_block_with_more_keys_than_16_bit_positions_hold(lib):
    """One node that every key reaches (a hub column of Psi) gives the first block a key list of N > 65535 entries:
    the build then looks positions up per row instead of keeping them in 16 bits, takes many accumulator passes for
    that block and walks a row of Psi^T far longer than its batched fetches.  Mask rows and attention against the oracle."""
    api, B, ctx = lib
    N, R = 66000, 66000
    rng = np.random.default_rng(4)
    # Phi: the diagonal plus, for the first rows, the hub node 0;  Psi: the diagonal plus the hub for every row
    pr, pc, pv = [0], [], []
    for i in range(N):
        cols = [0, i] if (0 < i < 40) else [i]
        pc += cols; pv += list(rng.uniform(0.5, 1.0, len(cols))); pr.append(len(pc))
    sr, sc, sv = [0], [], []
    for j in range(N):
        cols = [0, j] if j > 0 else [0]
        sc += cols; sv += list(rng.uniform(0.5, 1.0, len(cols))); sr.append(len(sc))
    Phi = oracle.CSR(np.array(pr, np.int32), np.array(pc, np.int32), np.array(pv, np.float32), None, (N, R))
    Psi = oracle.CSR(np.array(sr, np.int32), np.array(sc, np.int32), np.array(sv, np.float32), None, (N, R))
    feat = api.features_from_csr(ctx, N, R, (Phi.rowptr, Phi.col, Phi.val), (Psi.rowptr, Psi.col, Psi.val))
    B.grf_features_materialise(ctx.handle, feat.handle)
    B.grf_ctx_check(ctx.handle)
    rows = [0, 1, 17, 39, 40, 127, 128, 4095, N - 1]
    _check_mask(_mask_rows(B, ctx, feat, rows, N), oracle.mask_rows(Phi, Psi, rows), "hub column")
    q, k, v = tensors.qkv(1, N, 32, 64, "bf16", 5)
    out, den = api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda(), want_den=True)
    B.grf_ctx_check(ctx.handle)
    Mrows = oracle.mask_rows(Phi, Psi, rows)

    class _Rows:          # attn_bruteforce indexes the mask by absolute row
        def __getitem__(self, idx):
            return np.stack([Mrows[rows.index(int(r))] for r in np.atleast_1d(idx)])
    ref = oracle.attn_bruteforce(tensors.widen(q), tensors.widen(k), tensors.widen(v), _Rows(), rows=rows)
    helpers.assert_attn_close(out[:, rows].float().cpu().numpy(), ref, helpers.TOL["bf16"], den[:, rows].cpu().numpy(),
                              "hub column", same_sign=True)
    feat.free()


def test_host_buffer_path_over_the_mask_equals_device_calls(lib):
    """grf_step_host after grf_ctx_prefer_mask_route: same bits as sampling, materialising and calling the attention
    on device buffers; a shape the route does not cover falls back to the route through the per-node states."""
    api, B, ctx = lib
    w = configs.point_cloud_4096(1024)
    g = w.graph()
    f = B.grf_deconvolve(w.alpha).astype(np.float32)
    q, k, v = tensors.qkv(4, g.N, w.m, w.d, w.dtype, 3)
    out_h = torch.empty_like(v)
    B.grf_ctx_prefer_mask_route(ctx.handle, True)
    try:
        B.grf_step_host(ctx.handle, g.N, g.rowptr, g.col, g.w, 9, w.n_walks, w.p_halt, w.max_len, f, None,
                        4, w.m, w.d, B.GRF_DTYPE_BF16, q, k, v, out_h)
        feat = api.sample(ctx, api.DeviceGraph(g), 9, w.n_walks, w.p_halt, w.max_len, f)
        B.grf_features_materialise(ctx.handle, feat.handle)
        out_d = api.masked_attn_mhat(ctx, feat, q.cuda(), k.cuda(), v.cuda())
        assert torch.equal(out_h, out_d.cpu())
        # m = 8 is not covered by the mask route: the call must still work (per-node states)
        q8, k8, _ = tensors.qkv(4, g.N, 8, w.d, w.dtype, 3)
        out8 = torch.empty_like(v)
        B.grf_step_host(ctx.handle, g.N, g.rowptr, g.col, g.w, 9, w.n_walks, w.p_halt, w.max_len, f, None,
                        4, 8, w.d, B.GRF_DTYPE_BF16, q8, k8, v, out8)
        out8_d = api.masked_linear_attn(ctx, feat, q8.cuda(), k8.cuda(), v.cuda())
        assert torch.equal(out8, out8_d.cpu())
        feat.free()
    finally:
        B.grf_ctx_prefer_mask_route(ctx.handle, False)
