"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs."""
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
    ctx.close()


WALK_CASES = {
    "tiny": lambda: configs.tiny(),
    "vit": lambda: configs.vit_grid(),
    "pc1024": lambda: configs.point_cloud_4096(1024),
    "reg4096": lambda: configs.sweep(12),
}


@pytest.mark.parametrize("name", list(WALK_CASES))
def test_walks_bit_exact(lib, name):
    api, B, ctx = lib
    w = WALK_CASES[name]()
    g = w.graph()
    dg = api.DeviceGraph(g)
    shape = (2, g.N, w.n_walks, w.max_len + 1)
    traj = torch.empty(shape, dtype=torch.int32, device="cuda")
    load = torch.empty(shape, dtype=torch.float32, device="cuda")
    B.grf_debug_walks(ctx.handle, g.N, dg.rowptr, dg.col, dg.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len,
                      traj, load)
    torch.cuda.synchronize()
    o_traj, o_load = oracle.walks(g.rowptr, g.col, g.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len)
    assert np.array_equal(traj.cpu().numpy(), o_traj)
    assert np.array_equal(load.cpu().numpy().view(np.uint32), o_load.view(np.uint32))


@pytest.mark.parametrize("name", list(WALK_CASES))
def test_features_structure_bit_exact_values_close(lib, name):
    api, B, ctx = lib
    w = WALK_CASES[name]()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f)
    helpers.assert_csr_equal(feat.to_host(0), Phi, "Phi")
    helpers.assert_csr_equal(feat.to_host(1), Psi, "Psi")
    helpers.assert_csr_equal(feat.to_host(2), PsiT, "Psi^T")
    # same summation order on both sides: the fp32 values agree to the bit
    assert np.array_equal(feat.to_host(0)[2].view(np.uint32), Phi.val.view(np.uint32))
    # run-to-run determinism, reusing the same feature object
    before = [a.copy() for a in feat.to_host(2)]
    api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f, features=feat)
    after = feat.to_host(2)
    assert all(np.array_equal(a, b) for a, b in zip(before, after))
    feat.free()


def _attn_case(lib, w, g, G, f_phi=None, f_psi=None, ws_bytes=None, same_sign=False):
    api, B, ctx = lib
    if f_phi is None:
        f_phi = oracle.deconvolve(w.alpha).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
    q, k, v = tensors.qkv(G, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f_phi, f_psi)
    ref = oracle.attn_sparse(tensors.widen(q), tensors.widen(k), tensors.widen(v), Phi, PsiT)
    outs = []
    for tensor_cores in ((True, False) if w.dtype == "bf16" else (True,)):   # both gather kernels for bf16
        B.grf_ctx_use_tensor_cores(ctx.handle, tensor_cores)
        out, den = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda(), want_den=True,
                                          workspace_bytes=ws_bytes)
        B.grf_ctx_check(ctx.handle)
        helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL[w.dtype], den.cpu().numpy(),
                                  f"{w.name} tensor_cores={tensor_cores}", same_sign=same_sign)
        outs.append(out)
    B.grf_ctx_use_tensor_cores(ctx.handle, True)
    feat.free()
    return outs[0]


def test_attention_tiny_fp32(lib):
    w = configs.tiny()
    _attn_case(lib, w, w.graph(), 1, same_sign=True)


def test_attention_vit_bf16(lib):
    w = configs.vit_grid()
    _attn_case(lib, w, w.graph(), 12)


def test_attention_point_cloud_bf16(lib):
    w = configs.point_cloud_4096(2048)
    _attn_case(lib, w, w.graph(), 2, same_sign=True)


def test_attention_regular_graph_bf16(lib):
    w = configs.sweep(11)
    _attn_case(lib, w, w.graph(), 2, same_sign=True)


def test_attention_asymmetric_features(lib):
    """f_psi = delta_0: Psi = I (App. 'Asymmetric graph random features'), f_phi = alpha."""
    w = configs.tiny()
    f_psi = np.zeros(w.max_len + 1, np.float32); f_psi[0] = 1.0
    _attn_case(lib, w, w.graph(), 2, f_phi=w.alpha.astype(np.float32), f_psi=f_psi)


def test_attention_chunked_workspace_matches_single_pass(lib):
    api, B, ctx = lib
    w = configs.vit_grid()
    g = w.graph()
    per = B.grf_attn_workspace_bytes(1, g.N, w.m, w.d, B.GRF_DTYPE_BF16)
    a = _attn_case(lib, w, g, 5, ws_bytes=2 * per)     # chunks of 2, 2, 1
    b = _attn_case(lib, w, g, 5)
    assert torch.equal(a, b)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("m,d", [(8, 8), (16, 128), (128, 16), (64, 64), (32, 64), (128, 128), (16, 16), (64, 32)])
def test_attention_shapes_random_features(lib, m, d, dtype):
    """Rectangular (N x R), signed features: catches index or operand mix-ups for every tile shape."""
    api, B, ctx = lib
    rng = np.random.default_rng(m * 1000 + d)
    N, R, G = 331, 141, 3       # three query blocks of the tensor-core kernel, the last one ragged

    def rand_csr(rows, cols, per_row):
        rowptr = [0]; col = []; val = []
        for r in range(rows):
            # rows 0, 5, 130 and the last one (one in every query block, the ragged one included) and about one in
            # ten of the others have no entry at all: Eq. 12 with an empty sum, out = 0
            n = 0 if r in (0, 5, 130, rows - 1) else rng.integers(0, per_row + 1) * (rng.random() > 0.1)
            c = np.sort(rng.choice(cols, size=n, replace=False))
            col += list(c); val += list(rng.standard_normal(len(c))); rowptr.append(len(col))
        return oracle.CSR(np.array(rowptr, np.int32), np.array(col, np.int32), np.array(val, np.float32), None, (rows, cols))

    Phi, Psi = rand_csr(N, R, 9), rand_csr(N, R, 12)
    assert (np.diff(Phi.rowptr) == 0).sum() >= 4
    feat = api.features_from_csr(ctx, N, R, (Phi.rowptr, Phi.col, Phi.val), (Psi.rowptr, Psi.col, Psi.val))
    PsiT = oracle.transpose(Psi)
    helpers.assert_csr_equal(feat.to_host(2), PsiT, "Psi^T", val_rtol=0)
    q, k, v = tensors.qkv(G, N, m, d, dtype, 5)
    ref = oracle.attn_sparse(tensors.widen(q), tensors.widen(k), tensors.widen(v), Phi, PsiT)
    for tensor_cores in ((True, False) if dtype == "bf16" else (True,)):
        B.grf_ctx_use_tensor_cores(ctx.handle, tensor_cores)
        out, den = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda(), want_den=True)
        B.grf_ctx_check(ctx.handle)
        helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL[dtype], den.cpu().numpy(),
                                  f"m{m} d{d} tensor_cores={tensor_cores}")
    B.grf_ctx_use_tensor_cores(ctx.handle, True)
    feat.free()


@pytest.mark.parametrize("m,d", [(16, 64), (32, 64), (64, 64), (32, 32)])
def test_state_kernels_key_count_edges(lib, m, d):
    """Nodes with 0, 1, 15 ... 200 keys: empty items, items that end on and next to the 16-key steps and the
    64-key item boundary, nodes of several items; more than 64 nodes, so that two CTAs share the work."""
    api, B, ctx = lib
    rng = np.random.default_rng(7 * m + d)
    N, G = 256, 2
    lengths = [0, 1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 200] * 6      # R = 72 nodes
    R = len(lengths)
    cols_of_node = [np.sort(rng.choice(N, size=c, replace=False)) for c in lengths]
    rows = [[] for _ in range(N)]
    for l, js in enumerate(cols_of_node):
        for j in js:
            rows[j].append(l)
    rowptr = np.zeros(N + 1, np.int32); col = []; val = []
    for j in range(N):
        col += rows[j]; val += list(rng.uniform(0.1, 1.0, len(rows[j]))); rowptr[j + 1] = len(col)
    Psi = oracle.CSR(rowptr, np.array(col, np.int32), np.array(val, np.float32), None, (N, R))
    prow = [0]; pcol = []; pval = []
    for _ in range(N):
        c = np.sort(rng.choice(R, size=rng.integers(1, 8), replace=False))
        pcol += list(c); pval += list(rng.uniform(0.1, 1.0, len(c))); prow.append(len(pcol))
    Phi = oracle.CSR(np.array(prow, np.int32), np.array(pcol, np.int32), np.array(pval, np.float32), None, (N, R))
    feat = api.features_from_csr(ctx, N, R, (Phi.rowptr, Phi.col, Phi.val), (Psi.rowptr, Psi.col, Psi.val))
    PsiT = oracle.transpose(Psi)
    assert list(np.diff(PsiT.rowptr)) == lengths
    q, k, v = tensors.qkv(G, N, m, d, "bf16", 11)
    ref = oracle.attn_sparse(tensors.widen(q), tensors.widen(k), tensors.widen(v), Phi, PsiT)
    out, den = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda(), want_den=True)
    B.grf_ctx_check(ctx.handle)
    helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL["bf16"], den.cpu().numpy(), f"key edges m{m} d{d}",
                              same_sign=True)
    feat.free()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("softmax", [False, True])
def test_asymmetric_attention_matches_oracle(lib, dtype, softmax):
    """Alg. 2: features sampled with f_psi = delta_0; the fused kernel against the dense definition with
    Mhat = Phi, and (linear kernel) against the general S/z path on the same feature object."""
    api, B, ctx = lib
    w = configs.point_cloud_4096(1024)
    g = w.graph()
    f_phi = w.alpha.astype(np.float32)
    f_psi = np.zeros(w.max_len + 1, np.float32); f_psi[0] = 1.0
    feat = api.sample(ctx, api.DeviceGraph(g), configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
    Phi, Psi, PsiT, _, _ = helpers.oracle_features(w, g, configs.WALK_SEED, f_phi, f_psi)
    G = 3
    q, k, v = tensors.qkv(G, g.N, w.m, w.d, dtype, configs.QKV_SEED)
    if softmax:
        q = (q.float() * 0.25).to(q.dtype); k = (k.float() * 0.25).to(k.dtype)
    ref = oracle.attn_bruteforce(tensors.widen(q), tensors.widen(k), tensors.widen(v), Phi.dense(),
                                 kernel="exp" if softmax else "linear")
    out, den = api.masked_attn_asym(ctx, feat, q.cuda(), k.cuda(), v.cuda(), softmax=softmax, want_den=True)
    B.grf_ctx_check(ctx.handle)
    den_h = den.cpu().numpy()
    if softmax:     # the kernel's denominators are relative to exp(row maximum): compare the quotient only
        den_h = None
    helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL[dtype], den_h, f"asym softmax={softmax} {dtype}")
    if not softmax:
        general = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda())
        B.grf_ctx_check(ctx.handle)
        tol = 2e-2 if dtype == "bf16" else 1e-5
        assert torch.allclose(out.float(), general.float(), rtol=tol, atol=tol)
    # run-to-run identical
    again = api.masked_attn_asym(ctx, feat, q.cuda(), k.cuda(), v.cuda(), softmax=softmax)
    assert torch.equal(out, again)
    feat.free()


@pytest.mark.parametrize("m,d", [(8, 8), (16, 128), (128, 16), (64, 64), (32, 32)])
def test_asymmetric_attention_shapes(lib, m, d):
    api, B, ctx = lib
    rng = np.random.default_rng(m + 7 * d)
    N, G = 203, 2
    rowptr = [0]; col = []; val = []
    for i in range(N):
        c = np.sort(rng.choice(N, size=rng.integers(0, 70), replace=False))      # empty rows and rows of 3 batches
        col += list(c); val += list(rng.uniform(0.1, 1.0, len(c))); rowptr.append(len(col))
    Phi = oracle.CSR(np.array(rowptr, np.int32), np.array(col, np.int32), np.array(val, np.float32), None, (N, N))
    eye = (np.arange(N + 1, dtype=np.int32), np.arange(N, dtype=np.int32), np.ones(N, np.float32))
    feat = api.features_from_csr(ctx, N, N, (Phi.rowptr, Phi.col, Phi.val), eye)
    for dtype in ("fp32", "bf16"):
        q, k, v = tensors.qkv(G, N, m, d, dtype, 3)
        for softmax in (False, True):
            qq, kk = (q, k) if not softmax else ((q.float() * 0.2).to(q.dtype), (k.float() * 0.2).to(k.dtype))
            ref = oracle.attn_bruteforce(tensors.widen(qq), tensors.widen(kk), tensors.widen(v), Phi.dense(),
                                         kernel="exp" if softmax else "linear")
            out = api.masked_attn_asym(ctx, feat, qq.cuda(), kk.cuda(), v.cuda(), softmax=softmax)
            B.grf_ctx_check(ctx.handle)
            helpers.assert_attn_close(out.float().cpu().numpy(), ref, helpers.TOL[dtype], None, f"asym m{m} d{d} {dtype} softmax={softmax}")
    feat.free()


def test_identity_features_return_values(lib):
    api, B, ctx = lib
    N, G, m, d = 300, 2, 32, 64
    eye = (np.arange(N + 1, dtype=np.int32), np.arange(N, dtype=np.int32), np.ones(N, np.float32))
    feat = api.features_from_csr(ctx, N, N, eye, eye)
    q, k, v = tensors.qkv(G, N, m, d, "fp32", 1)
    q = q + 0.1; k = k + 0.1
    out = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    assert torch.allclose(out.cpu(), v, rtol=1e-5, atol=1e-6)
    feat.free()


def test_single_shared_column_is_unmasked_linear_attention(lib):
    """R = 1, all ones: Mhat = 1 1^T, i.e. Eq. 3, checked against an einsum in fp64."""
    api, B, ctx = lib
    N, G, m, d = 257, 2, 16, 32
    ones = (np.arange(N + 1, dtype=np.int32), np.zeros(N, np.int32), np.ones(N, np.float32))
    feat = api.features_from_csr(ctx, N, 1, ones, ones)
    q, k, v = tensors.qkv(G, N, m, d, "fp32", 2)
    out = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda()).cpu().numpy()
    qd, kd, vd = (t.numpy().astype(np.float64) for t in (q, k, v))
    num = np.einsum("gnm,gmd->gnd", qd, np.einsum("gnm,gnd->gmd", kd, vd))
    den = np.einsum("gnm,gm->gn", qd, kd.sum(axis=1))
    assert np.allclose(out, num / den[..., None], rtol=2e-4, atol=1e-5)
    feat.free()


def test_sampler_edge_cases(lib):
    api, B, ctx = lib
    # max_len = 0: only the zero-hop deposit, Phi = f_0 I
    g = graphs.grid_graph(5, 7, 0.25, False)
    dg = api.DeviceGraph(g)
    feat = api.sample(ctx, dg, 1, 3, 0.3, 0, np.array([0.75], np.float32))
    rp, c, v = feat.to_host(0)
    assert np.array_equal(rp, np.arange(36)) and np.array_equal(c, np.arange(35)) and np.allclose(v, 0.75)
    feat.free()
    # more walkers than lanes, p_halt = 0, zero coefficients, a graph with isolated and dangling nodes
    rowptr = np.array([0, 1, 2, 2, 4, 5, 6], np.int32)       # node 2 isolated
    col = np.array([1, 0, 4, 5, 3, 3], np.int32)
    wts = np.array([0.5, 0.5, 0.3, 0.2, 0.3, 0.2], np.float32)
    g2 = graphs.Graph(rowptr, col, wts)
    f = np.array([1.0, 0.0, 0.5, -0.25, 0.0, 0.125], np.float32)
    for n_walks, p in ((40, 0.0), (33, 0.2), (1, 0.5)):
        feat = api.sample(ctx, api.DeviceGraph(g2), 77, n_walks, p, 5, f)
        Phi, Psi, PsiT, _, _ = oracle.sample(g2.rowptr, g2.col, g2.w, 77, n_walks, p, 5, f)
        helpers.assert_csr_equal(feat.to_host(0), Phi, "Phi")
        helpers.assert_csr_equal(feat.to_host(2), PsiT, "Psi^T")
        feat.free()
    # long walks: capacity near the documented limit (n_walks * (max_len + 1) = 100 * 101)
    g3 = graphs.grid_graph(6, 6, 0.25, False)
    f3 = (0.7 ** np.arange(101)).astype(np.float32)
    feat = api.sample(ctx, api.DeviceGraph(g3), 5, 100, 0.1, 100, f3)
    Phi, Psi, PsiT, _, _ = oracle.sample(g3.rowptr, g3.col, g3.w, 5, 100, 0.1, 100, f3)
    helpers.assert_csr_equal(feat.to_host(0), Phi, "Phi long")
    helpers.assert_csr_equal(feat.to_host(1), Psi, "Psi long")
    feat.free()


def test_invalid_arguments_are_rejected_on_the_host(lib):
    api, B, ctx = lib
    g = graphs.grid_graph(4, 4, 0.25, False)
    dg = api.DeviceGraph(g)
    f = np.ones(3, np.float32)
    for kwargs, code in (
        (dict(n_walks=0), B.GRF_ERR_INVALID),
        (dict(p_halt=1.0), B.GRF_ERR_INVALID),
        (dict(p_halt=-0.1), B.GRF_ERR_INVALID),
        (dict(n_walks=20000), B.GRF_ERR_TOO_LARGE),
    ):
        args = dict(n_walks=2, p_halt=0.5)
        args.update(kwargs)
        with pytest.raises(B.GrfError) as ei:
            B.grf_sample(ctx.handle, g.N, dg.rowptr, dg.col, dg.w, 1, args["n_walks"], args["p_halt"], 2, f)
        assert ei.value.code == code
    with pytest.raises(B.GrfError):
        B.grf_sample(ctx.handle, 0, dg.rowptr, dg.col, dg.w, 1, 2, 0.5, 2, f)
    feat = api.sample(ctx, dg, 1, 2, 0.5, 2, f)
    q, k, v = tensors.qkv(1, g.N, 16, 16, "fp32", 0)
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    out = torch.empty_like(v, device="cuda")
    with pytest.raises(B.GrfError) as ei:
        B.grf_masked_linear_attn(ctx.handle, feat.handle, 1, g.N, 16, 16, 0, q.cuda(), k.cuda(), v.cuda(), out, None, ws, 1024)
    assert ei.value.code == B.GRF_ERR_WORKSPACE
    with pytest.raises(B.GrfError) as ei:   # unsupported feature dimension
        B.grf_masked_linear_attn(ctx.handle, feat.handle, 1, g.N, 12, 16, 0, q.cuda(), k.cuda(), v.cuda(), out, None, ws, 1024)
    assert ei.value.code == B.GRF_ERR_INVALID
    with pytest.raises(B.GrfError) as ei:   # N that does not match the features
        B.grf_masked_linear_attn(ctx.handle, feat.handle, 1, g.N + 1, 16, 16, 0, q.cuda(), k.cuda(), v.cuda(), out, None, ws, 1024)
    assert ei.value.code == B.GRF_ERR_INVALID
    feat.free()


def test_transpose_standalone(lib):
    api, B, ctx = lib
    w = configs.sweep(12)
    g = w.graph()
    # the graph itself is a handy sparse matrix; its transpose must equal the oracle's regrouping
    src = oracle.CSR(g.rowptr, g.col, g.w, None, (g.N, g.N))
    want = oracle.transpose(src)
    dg = api.DeviceGraph(g)
    t_rp = torch.empty(g.N + 1, dtype=torch.int32, device="cuda")
    t_c = torch.empty(g.E, dtype=torch.int32, device="cuda")
    t_v = torch.empty(g.E, dtype=torch.float32, device="cuda")
    B.grf_csr_transpose(ctx.handle, g.N, g.N, g.E, dg.rowptr, dg.col, dg.w, t_rp, t_c, t_v)
    torch.cuda.synchronize()
    helpers.assert_csr_equal((t_rp.cpu().numpy(), t_c.cpu().numpy(), t_v.cpu().numpy()), want, "transpose", val_rtol=0)


def test_transpose_columns_of_every_length_class(lib):
    """Columns with 0, a few, a few hundred (sorted in shared memory) and several thousand entries (sorted in place),
    rectangular, rows in arbitrary arrival order: the regrouped matrix must equal the oracle's, bit for bit."""
    api, B, ctx = lib
    rng = np.random.default_rng(11)
    rows, cols = 6000, 40
    want_len = [0, 1, 5, 31, 32, 33, 64, 100, 191, 192, 193, 200, 255, 256, 257, 500, 1000, 1023, 1024, 1025, 1500, 3000, 5999, 6000]
    want_len += [int(x) for x in rng.integers(0, 400, cols - len(want_len))]
    member = np.zeros((rows, cols), dtype=bool)
    for c, n in enumerate(want_len):
        member[rng.choice(rows, size=n, replace=False), c] = True
    rp = np.zeros(rows + 1, dtype=np.int32)
    rp[1:] = np.cumsum(member.sum(axis=1))
    ci = np.nonzero(member)[1].astype(np.int32)           # row-major order: columns ascending inside a row
    vals = rng.standard_normal(ci.size).astype(np.float32)
    nnz = int(ci.size)
    want = oracle.transpose(oracle.CSR(rp, ci, vals, None, (rows, cols)))
    d = lambda a: torch.from_numpy(a).cuda()
    t_rp = torch.empty(cols + 1, dtype=torch.int32, device="cuda")
    t_c = torch.empty(nnz, dtype=torch.int32, device="cuda")
    t_v = torch.empty(nnz, dtype=torch.float32, device="cuda")
    B.grf_csr_transpose(ctx.handle, rows, cols, nnz, d(rp), d(ci), d(vals), t_rp, t_c, t_v)
    torch.cuda.synchronize()
    helpers.assert_csr_equal((t_rp.cpu().numpy(), t_c.cpu().numpy(), t_v.cpu().numpy()), want, "transpose, all length classes",
                             val_rtol=0)


def test_step_host_matches_device_path(lib):
    api, B, ctx = lib
    w = configs.point_cloud_4096(512)
    g = w.graph()
    f = B.grf_deconvolve(w.alpha).astype(np.float32)
    q, k, v = tensors.qkv(2, g.N, w.m, w.d, w.dtype, 3)
    out_h = torch.empty_like(v)
    B.grf_step_host(ctx.handle, g.N, g.rowptr, g.col, g.w, 9, w.n_walks, w.p_halt, w.max_len, f, None,
                    2, w.m, w.d, B.GRF_DTYPE_BF16, q, k, v, out_h)
    feat = api.sample(ctx, api.DeviceGraph(g), 9, w.n_walks, w.p_halt, w.max_len, f)
    out_d = api.masked_linear_attn(ctx, feat, q.cuda(), k.cuda(), v.cuda())
    assert torch.equal(out_h, out_d.cpu())
    feat.free()
    bad = g.col.copy(); bad[0] = g.N
    with pytest.raises(B.GrfError) as ei:
        B.grf_step_host(ctx.handle, g.N, g.rowptr, bad, g.w, 9, w.n_walks, w.p_halt, w.max_len, f, None,
                        2, w.m, w.d, B.GRF_DTYPE_BF16, q, k, v, out_h)
    assert ei.value.code == B.GRF_ERR_BADGRAPH


def test_deconvolve_matches_oracle(lib):
    api, B, ctx = lib
    for w in (configs.tiny(), configs.vit_grid()):
        assert np.allclose(B.grf_deconvolve(w.alpha), oracle.deconvolve(w.alpha), rtol=1e-14, atol=0)


def test_device_graph_check_rejects_inconsistent_graphs(lib):
    """With grf_ctx_check_graphs on, a device-resident graph is validated by a kernel before any walk: a
    decreasing row pointer, a column index out of range and a non-zero first row pointer are all refused."""
    api, B, ctx = lib
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    B.grf_ctx_check_graphs(ctx.handle, True)
    try:
        good = api.sample(ctx, api.DeviceGraph(g), 1, w.n_walks, w.p_halt, w.max_len, f)
        good.free()
        for kind in ("rowptr_decreases", "col_too_large", "col_negative", "rowptr0"):
            dg = api.DeviceGraph(g)
            if kind == "rowptr_decreases":
                dg.rowptr[5] = dg.rowptr[4] - 1
            elif kind == "col_too_large":
                dg.col[7] = g.N
            elif kind == "col_negative":
                dg.col[3] = -2
            else:
                dg.rowptr[0] = 1
            with pytest.raises(B.GrfError) as e:
                api.sample(ctx, dg, 1, w.n_walks, w.p_halt, w.max_len, f)
            assert e.value.code == B.GRF_ERR_BADGRAPH, kind
    finally:
        B.grf_ctx_check_graphs(ctx.handle, False)
    B.grf_ctx_check(ctx.handle)


def test_bounded_wait_gives_up_and_reports_timeout(lib):
    """A wait for a barrier that nothing arrives at runs out after its limit (here about a millisecond), the error
    word is raised, grf_ctx_check reports GRF_ERR_TIMEOUT once, and the context keeps working afterwards."""
    api, B, ctx = lib
    B.grf_ctx_check(ctx.handle)
    B.grf_debug_wait_timeout(ctx.handle, 2_000_000)
    with pytest.raises(B.GrfError) as e:
        B.grf_ctx_check(ctx.handle)
    assert e.value.code == B.GRF_ERR_TIMEOUT
    B.grf_ctx_check(ctx.handle)                       # the word was cleared
    w = configs.tiny()
    _attn_case(lib, w, w.graph(), 1, same_sign=True)   # and the device is as usable as before
    B.grf_ctx_check(ctx.handle)
