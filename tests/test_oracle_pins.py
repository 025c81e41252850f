"""Pins for the CPU oracle: each test ties a part of oracle/ to something fixed by the paper or
by mathematics (known answers, closed forms, library routines, brute force), not to the oracle
itself.  No GPU needed."""
import os
from math import comb

import numpy as np
import pytest
import scipy.sparse as sp

import oracle
from workloads import configs, graphs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        return [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]


# ------------------------------------------------------------------ Philox

def test_philox_known_answers():
    for row in _golden_rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in row]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_philox_counter_and_key_sensitivity():
    base = oracle.philox4x32_10((1, 2, 3, 4), (5, 6))
    seen = {tuple(base)}
    for pos in range(4):
        c = [1, 2, 3, 4]; c[pos] += 1
        seen.add(tuple(oracle.philox4x32_10(c, (5, 6))))
    for pos in range(2):
        k = [5, 6]; k[pos] += 1
        seen.add(tuple(oracle.philox4x32_10((1, 2, 3, 4), k)))
    assert len(seen) == 7


# ------------------------------------------------------------------ Remark 3.1 and Eq. 4

def test_deconvolve_closed_form_geometric():
    want = np.array([float(r[0]) for r in _golden_rows("deconvolution_geometric.txt")])
    got = oracle.deconvolve(0.5 ** np.arange(len(want)))
    assert np.allclose(got, want, rtol=0, atol=1e-16)
    assert np.allclose(want, [comb(2 * k, k) / 8 ** k for k in range(len(want))], rtol=0, atol=0)


def test_deconvolve_convolution_identity_random_alpha():
    rng = np.random.default_rng(0)
    for _ in range(20):
        a = rng.random(11); a[0] += 0.25
        f = oracle.deconvolve(a)
        assert np.allclose(np.convolve(f, f)[:11], a, rtol=0, atol=1e-12)


def test_power_series_against_matrix_inverse():
    """sum_k (W/2)^k = (I - W/2)^-1 (Neumann series) on the 8x8 grid, whose spectral radius is < 1."""
    W = graphs.grid_graph(8, 8, 0.25, False).dense()
    got = oracle.power_series(W, 0.5 ** np.arange(200))
    want = np.linalg.inv(np.eye(64) - 0.5 * W)
    assert np.abs(got - want).max() < 1e-13
    # the truncated mask of the tiny workload is close to, but not equal to, the infinite series
    trunc = oracle.power_series(W, 0.5 ** np.arange(9))
    assert 1e-6 < np.abs(trunc - want).max() < 1e-3


def test_feature_factorisation_of_mask():
    """Remark 3.1 with truncation: F_L F_L^T = sum_{k<=2L} (f*f)_k W^k; its first L+1 coefficients are alpha."""
    W = graphs.grid_graph(8, 8, 0.25, False).dense()
    alpha = 0.5 ** np.arange(9)
    f = oracle.deconvolve(alpha)
    F = oracle.power_series(W, f)
    conv = np.convolve(f, f)
    assert np.allclose(conv[:9], alpha, atol=1e-15)
    assert np.abs(F @ F.T - oracle.power_series(W, conv)).max() < 1e-14
    assert np.abs(F - F.T).max() < 1e-15  # W symmetric
    # distance of the estimator's target from the truncated alpha series (left-over terms k > L)
    assert 1e-6 < np.abs(F @ F.T - oracle.power_series(W, alpha)).max() < 2e-4


# ------------------------------------------------------------------ walks

def _sample_tiny(seed, n=4, p=0.5, L=8):
    g = graphs.grid_graph(8, 8, 0.25, False)
    return g, oracle.walks(g.rowptr, g.col, g.w, seed, n, p, L)


def test_trajectories_follow_edges_and_start_at_source():
    g, (traj, load) = _sample_tiny(3)
    W = g.dense()
    assert (traj[:, :, :, 0] == np.arange(64)[None, :, None]).all()
    assert (load[:, :, :, 0] == 1.0).all()
    ended = traj < 0
    assert (ended[..., 1:] >= ended[..., :-1]).all()       # once ended, stays ended
    a, b = traj[..., :-1], traj[..., 1:]
    ok = b >= 0
    assert (W[a[ok], b[ok]] > 0).all()
    assert (load[ended] == 0).all()


def test_load_is_importance_weight_of_prefix():
    """load_t = prod_hops W_uv * deg(u) / (1 - p): Eq. 9 over p(omega) of a simple random walk that
    survives each hop with probability 1 - p.  Recomputed in fp64 from the trajectory."""
    w = configs.point_cloud_4096(256)
    g = w.graph()
    traj, load = oracle.walks(g.rowptr, g.col, g.w, 11, 8, 0.1, 12)
    W = sp.csr_matrix((g.w.astype(np.float64), g.col, g.rowptr), shape=(g.N, g.N))
    deg = np.diff(g.rowptr)
    rng = np.random.default_rng(0)
    for _ in range(300):
        e, i, k = rng.integers(2), rng.integers(g.N), rng.integers(8)
        want = 1.0
        for t in range(1, 13):
            if traj[e, i, k, t] < 0:
                break
            u, v = traj[e, i, k, t - 1], traj[e, i, k, t]
            want *= W[u, v] * deg[u] / (1.0 - np.float32(0.1).astype(np.float64))
            assert abs(load[e, i, k, t] - want) <= 1e-5 * want


def test_deterministic_walks_on_perfect_matching():
    """All degrees 1 and p_halt = 0: every walk is the same, so Phi equals F_L(W) for every seed."""
    g = graphs.perfect_matching_graph(10, 0.7)
    W = g.dense()
    f = np.array([1.0, 0.5, -0.25, 0.125, 0.0, 0.3], dtype=np.float32)
    F = oracle.power_series(W, f.astype(np.float64))
    for seed in (0, 1, 99):
        Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, seed, 3, 0.0, 5, f)
        assert np.abs(Phi.dense() - F).max() < 1e-6
        assert np.abs(Psi.dense() - F).max() < 1e-6
        assert np.array_equal(PsiT.dense(), Psi.dense().T)
        assert np.abs(Phi.val.astype(np.float64) - Phi.val64).max() < 1e-6


def test_walk_length_distribution_geometric():
    """Halting coin before every hop: P(>= k hops) = (1-p)^k for k <= L; the number of visited nodes
    per walk has mean (1 - (1-p)^(L+1)) / p on a graph without dead ends."""
    g = graphs.random_regular_graph(512, 5)
    for p, L in ((0.5, 8), (0.1, 12), (0.15, 10)):
        traj, _ = oracle.walks(g.rowptr, g.col, g.w, 123, 16, p, L)
        hops = (traj >= 0).sum(axis=-1).ravel() - 1
        n = hops.size
        for k in range(1, L + 1):
            q = (1 - np.float32(p).astype(np.float64)) ** k
            frac = (hops >= k).mean()
            assert abs(frac - q) < 4.5 * np.sqrt(q * (1 - q) / n) + 1e-9, (p, k)
        mean_visits = (hops + 1).mean()
        want = (1 - (1 - p) ** (L + 1)) / p
        assert abs(mean_visits - want) < 0.02 * want


def test_neighbour_choice_uniform():
    g = graphs.grid_graph(8, 8, 0.25, False)
    counts = np.zeros((64, 64))
    for seed in range(40):
        traj, _ = oracle.walks(g.rowptr, g.col, g.w, seed, 64, 0.0, 1)
        a, b = traj[..., 0].ravel(), traj[..., 1].ravel()
        np.add.at(counts, (a, b), 1)
    deg = np.diff(g.rowptr)
    total = counts.sum(axis=1)
    for i in range(64):
        nb = g.col[g.rowptr[i]:g.rowptr[i + 1]]
        expect = total[i] / deg[i]
        chi2 = ((counts[i, nb] - expect) ** 2 / expect).sum()
        assert chi2 < 25.0, (i, chi2)   # chi-square with <= 3 dof; 25 is far in the tail
        assert counts[i].sum() == counts[i, nb].sum()


def test_ensembles_are_independent_streams():
    _, (traj, _) = _sample_tiny(5, n=8, p=0.1, L=8)
    assert not np.array_equal(traj[0], traj[1])
    _, (traj2, _) = _sample_tiny(6, n=8, p=0.1, L=8)
    assert not np.array_equal(traj[0], traj2[0])
    _, (traj3, _) = _sample_tiny(5, n=8, p=0.1, L=8)
    assert np.array_equal(traj, traj3)
    # a seed that differs only in its high 32 bits is a different stream
    g = graphs.grid_graph(8, 8, 0.25, False)
    t_hi, _ = oracle.walks(g.rowptr, g.col, g.w, 5 + (1 << 32), 8, 0.1, 8)
    assert not np.array_equal(traj, t_hi)


def test_feature_l1_norm_bounded_by_c():
    """Proof of Thm 3.2: every walk deposits at most c = sum_k |f_k| (max W_ij d_i / (1-p))^k in L1,
    so each feature row (a mean over n walks) has L1 norm <= c; the diagonal holds exactly f_0."""
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    c = sum(abs(float(f[k])) * (0.25 * 4 / 0.5) ** k for k in range(9))
    assert abs(c - 3.3385) < 1e-3
    for seed in range(20):
        Phi, Psi, _, _, _ = oracle.sample(g.rowptr, g.col, g.w, seed, w.n_walks, w.p_halt, w.max_len, f)
        for M in (Phi, Psi):
            l1 = np.add.reduceat(np.abs(M.val64), M.rowptr[:-1])
            assert (l1 <= c + 1e-9).all()
            D = M.dense()
            assert (np.diag(D) >= f[0] - 1e-6).all()


def test_zero_coefficients_deposit_nothing():
    """f = delta_0 gives the identity (asymmetric GRFs, App. 'Asymmetric graph random features')."""
    g = graphs.grid_graph(8, 8, 0.25, False)
    f = np.zeros(9, dtype=np.float32); f[0] = 1.0
    Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, 1, 4, 0.5, 8, f)
    assert Phi.nnz == 64 and np.array_equal(Phi.col, np.arange(64))
    assert np.allclose(Phi.val, 1.0, atol=1e-6)


def test_row_sums_on_stochastic_graph():
    """E[sum_q Phi_iq] = sum_t f_t (W^t 1)_i; with W 1 = 1 (8-regular, weights 1/8) it is sum_t f_t
    for walks that cannot die early except by the coin."""
    w = configs.sweep(10)
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    Phi, Psi, _, _, _ = oracle.sample(g.rowptr, g.col, g.w, 42, w.n_walks, w.p_halt, w.max_len, f)
    want = float(f.astype(np.float64).sum())
    for M in (Phi, Psi):
        rs = np.add.reduceat(M.val64, M.rowptr[:-1])
        sem = rs.std() / np.sqrt(rs.size)
        assert abs(rs.mean() - want) < 4 * sem


def test_lemma_3_3_sparsity_bound():
    """With probability >= 1 - delta a feature has at most n*b nonzeros, b solving (1-(1-p)^b)^n = 1-delta."""
    w = configs.sweep(11)
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    Phi, _, _, _, _ = oracle.sample(g.rowptr, g.col, g.w, 1, w.n_walks, w.p_halt, w.max_len, f)
    nnz_row = np.diff(Phi.rowptr)
    n, p = w.n_walks, w.p_halt
    for delta in (0.5, 0.1, 0.01):
        b = np.log(1 - (1 - delta) ** (1 / n)) / np.log(1 - p)
        assert (nnz_row > n * b).mean() <= delta
    assert nnz_row.max() <= n * (w.max_len + 1)


@pytest.mark.parametrize("asym", [False, True])
def test_unbiasedness_monte_carlo(asym):
    """E[Phi] = F_L(W) and E[Phi Psi^T] = F_L G_L^T for independent ensembles (Sec. 3.3), over 10^4 seeds
    of the tiny workload.  Entries with enough non-zero samples are z-tested; the rest through sums."""
    w = configs.tiny()
    g = w.graph()
    W = g.dense()
    if asym:
        f_phi = w.alpha.astype(np.float32)
        f_psi = np.zeros(9, dtype=np.float32); f_psi[0] = 1.0
    else:
        f_phi = f_psi = oracle.deconvolve(w.alpha).astype(np.float32)
    F = oracle.power_series(W, f_phi.astype(np.float64))
    Gm = oracle.power_series(W, f_psi.astype(np.float64))
    target = F @ Gm.T
    if asym:
        assert np.abs(target - oracle.power_series(W, w.alpha)).max() < 1e-12
    S = 10000
    sumM = np.zeros((64, 64)); sumM2 = np.zeros((64, 64)); hits = np.zeros((64, 64))
    sumF = np.zeros((64, 64)); sumF2 = np.zeros((64, 64)); hitsF = np.zeros((64, 64))
    for seed in range(S):
        Phi, Psi, _, _, _ = oracle.sample(g.rowptr, g.col, g.w, seed, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
        P, Q = Phi.dense(), Psi.dense()
        M = P @ Q.T
        sumM += M; sumM2 += M * M; hits += M != 0
        sumF += P; sumF2 += P * P; hitsF += P != 0
    for mean, sq, cnt, want in ((sumM / S, sumM2 / S, hits, target), (sumF / S, sumF2 / S, hitsF, F)):
        sd = np.sqrt(np.maximum(sq - mean ** 2, 0))
        sel = cnt >= 200
        z = (mean[sel] - want[sel]) / (sd[sel] / np.sqrt(S))
        assert sel.sum() > 300
        assert np.abs(z).max() < 5.0
        assert (np.abs(z) > 3).mean() < 0.01
        # aggregates cover the rarely-hit entries
        row_err = mean.sum(axis=1) - want.sum(axis=1)
        row_sem = np.sqrt(sq.sum(axis=1) * 64) / np.sqrt(S)   # crude upper bound on the row-sum s.e.
        assert (np.abs(row_err) < 4 * row_sem).all()
        assert abs(mean.sum() / want.sum() - 1) < 5e-3


# ------------------------------------------------------------------ transpose

def test_transpose_matches_scipy():
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    _, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, 9, 4, 0.5, 8, f)
    ref = sp.csr_matrix((Psi.val, Psi.col, Psi.rowptr), shape=Psi.shape).T.tocsr()
    ref.sort_indices()
    assert np.array_equal(ref.indptr, PsiT.rowptr)
    assert np.array_equal(ref.indices, PsiT.col)
    assert np.array_equal(ref.data, PsiT.val)


# ------------------------------------------------------------------ attention

def _rand_csr(rng, rows, cols, per_row, signed=False):
    rowptr = [0]; col = []; val = []
    for _ in range(rows):
        k = rng.integers(0, per_row + 1)
        c = np.sort(rng.choice(cols, size=min(k, cols), replace=False))
        col += list(c)
        v = rng.standard_normal(len(c)) if signed else rng.random(len(c)) + 0.1
        val += list(v)
        rowptr.append(len(col))
    return oracle.CSR(np.array(rowptr, np.int32), np.array(col, np.int32), np.array(val, np.float32), None,
                      (rows, cols))


def _qkv(rng, G, N, m, d):
    q = np.maximum(rng.standard_normal((G, N, m)), 0).astype(np.float32)
    k = np.maximum(rng.standard_normal((G, N, m)), 0).astype(np.float32)
    v = rng.standard_normal((G, N, d)).astype(np.float32)
    return q, k, v


def test_bruteforce_against_scalar_loops():
    """Eqs. 1-2 spelled out with scalar loops on a tiny case with a NON-symmetric mask."""
    rng = np.random.default_rng(1)
    N, m, d = 5, 3, 2
    q, k, v = _qkv(rng, 1, N, m, d)
    q += 0.05; k += 0.05
    M = rng.random((N, N))
    got = oracle.attn_bruteforce(q, k, v, M)
    for i in range(N):
        num = [0.0] * d; den = 0.0
        for j in range(N):
            a = sum(float(q[0, i, s]) * float(k[0, j, s]) for s in range(m)) * M[i, j]
            den += a
            for b in range(d):
                num[b] += a * float(v[0, j, b])
        assert np.allclose(got["den"][0, i], den, rtol=1e-13)
        assert np.allclose(got["num"][0, i], num, rtol=1e-12, atol=1e-14)
        assert np.allclose(got["out"][0, i], np.array(num) / den, rtol=1e-12, atol=1e-14)


def test_sparse_route_equals_bruteforce_random_rectangular_features():
    """Eqs. 5-7: the S/z route equals Hadamard masking with Mhat = Phi Psi^T, for signed, non-square
    (N x R) features so that a transposed operand or swapped index cannot pass."""
    rng = np.random.default_rng(2)
    G, N, R, m, d = 2, 23, 17, 4, 6
    q, k, v = _qkv(rng, G, N, m, d)
    Phi = _rand_csr(rng, N, R, 5, signed=True)
    Psi = _rand_csr(rng, N, R, 4, signed=True)
    Mhat = Phi.dense() @ Psi.dense().T
    bf = oracle.attn_bruteforce(q, k, v, Mhat)
    sr = oracle.attn_sparse(q, k, v, Phi, oracle.transpose(Psi))
    assert np.allclose(sr["num"], bf["num"], rtol=1e-11, atol=1e-12)
    assert np.allclose(sr["den"], bf["den"], rtol=1e-11, atol=1e-12)
    assert (sr["num_abs"] >= np.abs(sr["num"]) - 1e-12).all()
    assert (sr["den_abs"] >= np.abs(sr["den"]) - 1e-12).all()


def test_sparse_route_equals_bruteforce_on_tiny_workload():
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, 42, w.n_walks, w.p_halt, w.max_len, f)
    rng = np.random.default_rng(3)
    q, k, v = _qkv(rng, 1, 64, 16, 16)
    bf = oracle.attn_bruteforce(q, k, v, Phi.dense() @ Psi.dense().T)
    sr = oracle.attn_sparse(q, k, v, Phi, PsiT)
    assert np.allclose(sr["out"], bf["out"], rtol=1e-10, atol=1e-12)
    rows = [0, 7, 63]
    assert np.allclose(oracle.mask_rows(Phi, Psi, rows), (Phi.dense() @ Psi.dense().T)[rows], atol=1e-15)


def _abs_inputs_reference(q, k, v, Phi, Psi):
    """The tolerance scale by its definition, computed densely: the sums of the absolute values of the terms of
    num and den are what Eqs. 1-2 give for |phi(q)|, |phi(k)|, |v| under the mask |Phi| |Psi|^T (every term of the
    S/z route is a product Phi_il q_a Psi_jl k_ja v_jb, so its absolute value factorises)."""
    Mabs = np.abs(Phi.dense()) @ np.abs(Psi.dense()).T
    return oracle.attn_bruteforce(np.abs(q), np.abs(k), np.abs(v), Mabs)


def test_tolerance_scale_nonnegative_features_equals_dense_definition():
    """num_abs / den_abs of the S/z route set the bound of every GPU comparison.  For non-negative features and
    phi(Q), phi(K) >= 0 every A_ij >= 0, so they must equal |A| |V| and sum_j |A_ij| of the dense definition."""
    w = configs.tiny()
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, 42, w.n_walks, w.p_halt, w.max_len, f)
    rng = np.random.default_rng(13)
    cases = [(Phi, Psi, 64, 16, 16, 1)]
    cases.append((_rand_csr(rng, 29, 11, 4, signed=False), _rand_csr(rng, 29, 11, 5, signed=False), 29, 5, 3, 2))
    for P, S, N, m, d, G in cases:
        assert (P.val >= 0).all() and (S.val >= 0).all()
        q, k, v = _qkv(rng, G, N, m, d)
        bf = oracle.attn_bruteforce(q, k, v, P.dense() @ S.dense().T)
        sr = oracle.attn_sparse(q, k, v, P, oracle.transpose(S))
        assert np.allclose(sr["num_abs"], bf["num_abs"], rtol=1e-11, atol=1e-300)
        assert np.allclose(sr["den_abs"], bf["den_abs"], rtol=1e-11, atol=1e-300)
        assert np.allclose(sr["den_abs"], sr["den"], rtol=1e-11, atol=1e-300)      # same-sign terms: no cancellation
        # and the definition itself: a term counted twice or squared would show here
        ab = _abs_inputs_reference(q, k, v, P, S)
        assert np.allclose(sr["num_abs"], ab["num"], rtol=1e-11, atol=1e-300)
        assert np.allclose(sr["den_abs"], ab["den"], rtol=1e-11, atol=1e-300)


def test_tolerance_scale_signed_features():
    """Signed rectangular features and signed phi: the scale equals the dense evaluation on absolute values
    exactly, and is never below the dense route's own |A| |V| (terms that cancel inside Mhat_ij count separately
    in the S/z route)."""
    rng = np.random.default_rng(14)
    G, N, R, m, d = 2, 31, 13, 4, 5
    q = rng.standard_normal((G, N, m)).astype(np.float32)
    k = rng.standard_normal((G, N, m)).astype(np.float32)
    v = rng.standard_normal((G, N, d)).astype(np.float32)
    Phi = _rand_csr(rng, N, R, 6, signed=True)
    Psi = _rand_csr(rng, N, R, 5, signed=True)
    sr = oracle.attn_sparse(q, k, v, Phi, oracle.transpose(Psi))
    ab = _abs_inputs_reference(q, k, v, Phi, Psi)
    # the S/z route sums |Phi_il q_a| * |Psi_jl k_ja v_jb| per feature component a; the dense evaluation on absolute
    # values sums (|q|.|k|) |Mhat|_ij |v_jb|: the same terms, regrouped
    assert np.allclose(sr["num_abs"], ab["num"], rtol=1e-11, atol=1e-300)
    assert np.allclose(sr["den_abs"], ab["den"], rtol=1e-11, atol=1e-300)
    bf = oracle.attn_bruteforce(q, k, v, Phi.dense() @ Psi.dense().T)
    assert (sr["num_abs"] >= bf["num_abs"] * (1 - 1e-12)).all()
    assert (sr["den_abs"] >= bf["den_abs"] * (1 - 1e-12)).all()
    assert (sr["num_abs"] > bf["num_abs"] * (1 + 1e-6)).any()        # and cancellation does occur in this case


def test_identity_features_return_values():
    """Phi = Psi = I: Mhat = I, so out_i = v_i wherever phi(q_i).phi(k_i) != 0."""
    rng = np.random.default_rng(4)
    G, N, m, d = 2, 12, 5, 7
    q, k, v = _qkv(rng, G, N, m, d)
    q += 0.1; k += 0.1
    eye = oracle.CSR(np.arange(N + 1, dtype=np.int32), np.arange(N, dtype=np.int32), np.ones(N, np.float32),
                     None, (N, N))
    out = oracle.attn_sparse(q, k, v, eye, oracle.transpose(eye))["out"]
    assert np.allclose(out, v, rtol=1e-12, atol=1e-12)


def test_all_ones_column_is_unmasked_linear_attention():
    """A single shared feature column (R = 1, all ones) gives Mhat = 1 1^T: Eq. 3, written as an einsum."""
    rng = np.random.default_rng(5)
    G, N, m, d = 2, 14, 4, 3
    q, k, v = _qkv(rng, G, N, m, d)
    ones = oracle.CSR(np.arange(N + 1, dtype=np.int32), np.zeros(N, np.int32), np.ones(N, np.float32), None, (N, 1))
    got = oracle.attn_sparse(q, k, v, ones, oracle.transpose(ones))
    kv = np.einsum("gnm,gnd->gmd", k.astype(np.float64), v.astype(np.float64))
    ksum = k.astype(np.float64).sum(axis=1)
    num = np.einsum("gnm,gmd->gnd", q.astype(np.float64), kv)
    den = np.einsum("gnm,gm->gn", q.astype(np.float64), ksum)
    assert np.allclose(got["num"], num, rtol=1e-12)
    assert np.allclose(got["den"], den, rtol=1e-12)


def test_asymmetric_route_equals_walk_accumulation():
    """Psi = I (f_psi = delta_0): Alg. 2 accumulates, over every prefix of every walk from v_i,
    phi(q_i).phi(k_j) * f_t * load * v_j with j the prefix's end node, then normalises."""
    w = configs.tiny()
    g = w.graph()
    f_phi = w.alpha.astype(np.float32)
    f_psi = np.zeros(9, np.float32); f_psi[0] = 1.0
    Phi, Psi, PsiT, traj, load = oracle.sample(g.rowptr, g.col, g.w, 7, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
    rng = np.random.default_rng(6)
    q, k, v = _qkv(rng, 1, 64, 16, 16)
    got = oracle.attn_sparse(q, k, v, Phi, PsiT)
    qd, kd, vd = q[0].astype(np.float64), k[0].astype(np.float64), v[0].astype(np.float64)
    for i in range(64):
        acc = np.zeros(16); s = 0.0
        for kk in range(w.n_walks):
            for t in range(9):
                j = traj[0, i, kk, t]
                if j < 0:
                    break
                a = float(qd[i] @ kd[j]) * float(f_phi[t]) * float(load[0, i, kk, t])
                acc += a * vd[j]; s += a
        assert np.allclose(got["out"][0, i], acc / s, rtol=1e-5, atol=1e-7)


# ----------------------------------------------------------------------------- asymmetric features (Alg. 2)

def test_softmax_kernel_with_all_ones_mask_is_plain_softmax_attention():
    """A = exp(QK^T) with the mask 1 everywhere is softmax attention: a library routine pins the exp branch."""
    from scipy.special import softmax
    rng = np.random.default_rng(3)
    Q = rng.standard_normal((2, 9, 5)) * 0.5; K = rng.standard_normal((2, 9, 5)) * 0.5; V = rng.standard_normal((2, 9, 4))
    got = oracle.attn_bruteforce(Q, K, V, np.ones((9, 9)), kernel="exp")["out"]
    want = np.stack([softmax(Q[g] @ K[g].T, axis=1) @ V[g] for g in range(2)])
    assert np.allclose(got, want, rtol=1e-12, atol=1e-14)


def test_asymmetric_route_three_ways():
    """Psi = I (f_psi = delta_0): the S/z route of Eq. 12, the dense definition with Mhat = Phi and the walk
    loop of Alg. 2 (which never forms Phi) give the same attention, for both similarity kernels where they apply."""
    w = configs.tiny()
    g = w.graph()
    f_phi = w.alpha.astype(np.float32)
    f_psi = np.zeros(w.max_len + 1, np.float32); f_psi[0] = 1.0
    Phi, Psi, PsiT, traj, load = oracle.sample(g.rowptr, g.col, g.w, 11, w.n_walks, w.p_halt, w.max_len, f_phi, f_psi)
    assert Psi.nnz == g.N and np.array_equal(Psi.col, np.arange(g.N)) and np.all(Psi.val == 1.0)
    rng = np.random.default_rng(5)
    f32 = lambda x: x.astype(np.float32).astype(np.float64)      # values that the fp32 interface of the S/z route keeps
    Q = f32(np.abs(rng.standard_normal((2, g.N, 6))) + 0.05); K = f32(np.abs(rng.standard_normal((2, g.N, 6))) + 0.05)
    V = f32(rng.standard_normal((2, g.N, 3)))
    dense = oracle.attn_bruteforce(Q, K, V, Phi.dense())["out"]
    sz = oracle.attn_sparse(Q, K, V, Phi, PsiT)["out"]
    walks = oracle.attn_asym_walks(Q, K, V, traj, load, f_phi)
    assert np.allclose(dense, sz, rtol=1e-10, atol=1e-12)
    assert np.allclose(dense, walks, rtol=1e-5, atol=1e-7)       # Phi's entries are fp32 sums of the walk terms
    dense_e = oracle.attn_bruteforce(Q * 0.3, K * 0.3, V, Phi.dense(), kernel="exp")["out"]
    walks_e = oracle.attn_asym_walks(Q * 0.3, K * 0.3, V, traj, load, f_phi, kernel="exp")
    assert np.allclose(dense_e, walks_e, rtol=1e-5, atol=1e-7)


# ------------------------------------------------------------------ re-modulation, FLOP counts, the mask itself

def test_keep_zero_structure_is_the_visited_set_and_values_agree_on_the_plain_support():
    """With keep_zero the index structure must not depend on f (it is the set of visited nodes), the values on the
    support of the plain assembly must be bit-identical to it, and the extra entries are exact zeros."""
    w = configs.tiny(); g = w.graph()
    traj, load = oracle.walks(g.rowptr, g.col, g.w, 5, w.n_walks, w.p_halt, w.max_len)
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    f[2] = 0.0; f[5] = 0.0
    plain = oracle.features_from_walks(traj, load, 0, f)
    kept = oracle.features_from_walks(traj, load, 0, f, keep_zero=True)
    ones = oracle.features_from_walks(traj, load, 0, np.ones_like(f), keep_zero=True)
    assert np.array_equal(kept.rowptr, ones.rowptr) and np.array_equal(kept.col, ones.col)
    # the visited set, straight from the trajectories
    for i in range(g.N):
        visited = np.unique(traj[0, i][traj[0, i] >= 0])
        assert np.array_equal(kept.col[kept.rowptr[i]:kept.rowptr[i + 1]], visited)
    assert kept.nnz > plain.nnz
    D = {(i, int(c)): v for i in range(g.N) for c, v in zip(kept.col[kept.rowptr[i]:kept.rowptr[i + 1]],
                                                             kept.val[kept.rowptr[i]:kept.rowptr[i + 1]])}
    on_plain = set()
    for i in range(g.N):
        for c, v in zip(plain.col[plain.rowptr[i]:plain.rowptr[i + 1]], plain.val[plain.rowptr[i]:plain.rowptr[i + 1]]):
            assert D[(i, int(c))].tobytes() == v.tobytes() or (D[(i, int(c))] == 0 and v == 0)
            on_plain.add((i, int(c)))
    assert all(v == 0 for key, v in D.items() if key not in on_plain)
    # no zero coefficient: the two assemblies are the same matrix
    f2 = oracle.deconvolve(w.alpha).astype(np.float32)
    a = oracle.features_from_walks(traj, load, 1, f2); b = oracle.features_from_walks(traj, load, 1, f2, keep_zero=True)
    assert np.array_equal(a.col, b.col) and a.val.tobytes() == b.val.tobytes()


def test_remodulation_is_linear_in_f():
    """Eq. 10 is linear in the coefficients: features(f) = sum_t f_t * features(e_t) (fp64 shadows, same walks)."""
    w = configs.tiny(); g = w.graph()
    traj, load = oracle.walks(g.rowptr, g.col, g.w, 11, w.n_walks, w.p_halt, w.max_len)
    rng = np.random.default_rng(3)
    f = rng.standard_normal(w.max_len + 1).astype(np.float32)
    full = oracle.features_from_walks(traj, load, 0, f, keep_zero=True)
    acc = np.zeros(full.nnz)
    for t in range(w.max_len + 1):
        e_t = np.zeros(w.max_len + 1, np.float32); e_t[t] = 1.0
        part = oracle.features_from_walks(traj, load, 0, e_t, keep_zero=True)
        assert np.array_equal(part.col, full.col)
        acc += float(f[t]) * part.val64
    assert np.allclose(acc, full.val64, rtol=1e-12, atol=1e-15)


def test_flop_counts_closed_forms_and_linear_growth():
    """Sec. 4 "Time complexity": 1-D grids, n = 4, p_halt = 0.5, m = d = 8, mean over 10 seeds.  The term-by-term
    count equals nnz * (m + 2m(d+1)) per matrix, stays below the bound from the expected number of deposits, grows
    linearly in N, and the softmax count grows quadratically."""
    m = d = 8; n = 4; p = 0.5; L = 8
    f = oracle.deconvolve(0.5 ** np.arange(L + 1)).astype(np.float32)
    means = {}
    for N in (64, 128, 256):
        g = graphs.path_graph(N, 0.5)
        counts = []
        for seed in range(10):
            Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, seed, n, p, L, f)
            c = oracle.flops_masked_linear(Phi, PsiT, m, d)
            assert c == (Phi.nnz + PsiT.nnz) * (m + 2 * m * (d + 1)) + N * d
            counts.append(c)
        means[N] = np.mean(counts)
        deposits = n * (1 - (1 - p) ** (L + 1)) / p          # expected deposits per row bound the row's non-zeros
        assert means[N] <= 2 * N * deposits * (m + 2 * m * (d + 1)) + N * d
        assert means[N] > oracle.flops_unmasked_linear(N, m, d)          # "a constant multiplicative cost"
    assert abs(means[128] / means[64] - 2) < 0.1 and abs(means[256] / means[128] - 2) < 0.1
    assert oracle.flops_unmasked_linear(128, m, d) == 4 * 128 * m * (d + 1) + 128 * d
    r = oracle.flops_softmax(256, m, d) / oracle.flops_softmax(128, m, d)
    assert 3.9 < r < 4.0


def test_materialised_mask_equals_dense_product():
    w = configs.tiny(); g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, 9, w.n_walks, w.p_halt, w.max_len, f)
    M = oracle.materialise(Phi, Psi)
    dense = Phi.dense() @ Psi.dense().T
    as64 = lambda X: sp.csr_matrix((X.val64, X.col, X.rowptr), shape=X.shape).toarray()
    assert np.allclose(as64(M), dense, rtol=0, atol=1e-15)
    assert np.allclose(M.dense(), dense, rtol=1e-7, atol=0)          # val is the fp32 rounding of val64
    ref = (sp.csr_matrix((np.ones(Phi.nnz), Phi.col, Phi.rowptr), shape=Phi.shape) @
           sp.csr_matrix((np.ones(Psi.nnz), Psi.col, Psi.rowptr), shape=Psi.shape).T).tocsr()
    ref.sort_indices()
    assert np.array_equal(M.rowptr, ref.indptr) and np.array_equal(M.col, ref.indices)      # structural support
    rows = [0, 7, 63]
    assert np.allclose(oracle.mask_rows(Phi, Psi, rows), dense[rows], rtol=0, atol=1e-15)
    # rectangular, signed
    rng = np.random.default_rng(2)
    A = sp.random(20, 13, 0.3, random_state=1, data_rvs=rng.standard_normal, format="csr"); A.sort_indices()
    Bm = sp.random(17, 13, 0.3, random_state=2, data_rvs=rng.standard_normal, format="csr"); Bm.sort_indices()
    a = oracle.CSR(A.indptr.astype(np.int32), A.indices.astype(np.int32), A.data.astype(np.float32), None, A.shape)
    b = oracle.CSR(Bm.indptr.astype(np.int32), Bm.indices.astype(np.int32), Bm.data.astype(np.float32), None, Bm.shape)
    M2 = oracle.materialise(a, b)
    assert M2.shape == (20, 17)
    assert np.allclose(as64(M2), a.dense() @ b.dense().T, rtol=0, atol=1e-12)
