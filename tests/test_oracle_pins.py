"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

The paper prints no worked numeric example, so the pins are closed forms, brute force on
tiny inputs, library routines of a different kind (a linear solve for an iteration's limit),
optimality conditions and invariants.  Each pin names the oracle function(s) it guards and
the mistake it would catch.
"""
import math
import os

import numpy as np
import pytest

from oracle import csat_oracle as orc
from oracle import phi_oracle as phi
from paper_2507_02957_b200 import workloads as wl

HERE = os.path.dirname(os.path.abspath(__file__))


# ----------------------------------------------------------------------------------------
# brute-force standard attention (the paper's Attn(Q,K,V) equation), pure Python loops
# ----------------------------------------------------------------------------------------
def brute_attention(Q, K, V, keys=None):
    nq, d = len(Q), len(Q[0])
    keys = list(range(len(K))) if keys is None else list(keys)
    out = [[0.0] * d for _ in range(nq)]
    for i in range(nq):
        s = []
        for j in keys:
            acc = 0.0
            for c in range(d):
                acc += Q[i][c] * K[j][c]
            s.append(acc / math.sqrt(d))
        mx = max(s)
        w = [math.exp(x - mx) for x in s]
        tot = sum(w)
        for c in range(d):
            acc = 0.0
            for t, j in enumerate(keys):
                acc += w[t] * V[j][c]
            out[i][c] = acc / tot
    return np.array(out)


def _rng(seed):
    return np.random.default_rng(seed)


# P1: m = n, Phi = I, recovery disabled  =>  standard softmax attention.
def test_identity_measurement_is_standard_attention():
    r = _rng(1)
    n, nq, d = 7, 5, 4
    Q, K, V = r.standard_normal((nq, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    out = orc.csat_forward_head(Q, K, V, np.eye(n), T=0, lam=0.1)
    ref = brute_attention(Q.tolist(), K.tolist(), V.tolist())
    assert np.abs(out - ref).max() <= 1e-12


# P1b: Phi = row-selection matrix  =>  standard attention restricted to the selected tokens.
# Catches a transposed or mis-indexed Phi, and Phi applied to the wrong axis.
def test_selection_measurement_is_attention_over_subset():
    r = _rng(2)
    n, nq, d = 9, 4, 3
    sel = [6, 0, 3, 7]
    Phi = np.zeros((len(sel), n))
    for row, j in enumerate(sel):
        Phi[row, j] = 1.0
    Q, K, V = r.standard_normal((nq, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    out = orc.csat_forward_head(Q, K, V, Phi, T=0, lam=0.0)
    ref = brute_attention(Q.tolist(), K.tolist(), V.tolist(), keys=sel)
    assert np.abs(out - ref).max() <= 1e-12


# Hand-sized closed forms.  m = 1: softmax over one measurement is 1, so Z = Phi V for every
# query; d = 1 makes every decoder quantity a scalar that can be written down.
def test_single_measurement_scalar_case_by_hand():
    a, b = 2.0, 1.0
    Phi = np.array([[a, b]])
    K = np.array([[0.7], [-1.3]])
    V = np.array([[3.0], [4.0]])
    Q = np.array([[0.2], [-5.0], [9.0]])
    Z = orc.csat_forward_head(Q, K, V, Phi, T=0, lam=0.1)
    assert np.allclose(Z, 10.0, atol=1e-14)           # 2*3 + 1*4
    # D = Phi[0,0] = 2, M = 2, G = 4, L = 4, mu = 1/4, S = 0, B = 1/2, theta = lambda/4
    out = orc.csat_forward_head(Q, K, V, Phi, T=3, lam=0.1)
    assert np.allclose(out, 10.0 / 2.0 - 0.1 / 4.0, atol=1e-14)   # soft(5, 0.025) = 4.975
    # a large threshold shrinks everything to zero
    out0 = orc.csat_forward_head(Q, K, V, Phi, T=3, lam=25.0)
    assert np.all(out0 == 0.0)


# m = 2, d = 1: softmax over two measurements is a logistic function of the score gap.
def test_two_measurements_logistic_closed_form():
    Phi = np.array([[1.0, 2.0, 0.0], [0.0, -1.0, 3.0]])
    K = np.array([[0.5], [0.25], [-1.0]])
    V = np.array([[1.0], [2.0], [4.0]])
    q = 1.5
    kt0, kt1 = 1.0 * 0.5 + 2.0 * 0.25, -0.25 - 3.0          # 1.0, -3.25
    vt0, vt1 = 1.0 + 4.0, -2.0 + 12.0                        # 5, 10
    p0 = 1.0 / (1.0 + math.exp(-(q * kt0 - q * kt1)))        # d = 1 -> scale 1
    z = p0 * vt0 + (1.0 - p0) * vt1
    Z = orc.csat_forward_head(np.array([[q]]), K, V, Phi, T=0, lam=0.0)
    assert abs(Z[0, 0] - z) <= 1e-13


# Q = 0  =>  uniform weights  =>  Z = mean over measurements of Phi V (any Phi).
def test_zero_queries_give_uniform_average():
    r = _rng(3)
    n, m, d = 10, 4, 3
    Phi, K, V = r.standard_normal((m, n)), r.standard_normal((n, d)), r.standard_normal((n, d))
    Z = orc.csat_forward_head(np.zeros((2, d)), K, V, Phi, T=0, lam=0.0)
    ref = np.zeros(d)
    for rr in range(m):
        for j in range(n):
            ref += Phi[rr, j] * V[j] / m
    assert np.abs(Z - ref[None, :]).max() <= 1e-13


# The scale argument and the default 1/sqrt(d): doubling d by zero-padding features changes only
# the scale, so scores with explicit scale must match.
def test_scale_is_inverse_sqrt_d():
    r = _rng(4)
    Q, Kt = r.standard_normal((3, 16)), r.standard_normal((5, 16))
    S = orc.compressed_scores(Q, Kt)
    for i in range(3):
        for rr in range(5):
            assert abs(S[i, rr] - sum(Q[i] * Kt[rr]) / 4.0) <= 1e-13


# P2: soft-threshold identities and its proximal definition.
def test_soft_threshold_identities_and_prox():
    x = np.linspace(-3, 3, 241)
    for theta in (0.0, 0.3, 1.0):
        s = orc.soft_threshold(x, theta)
        assert np.allclose(s, x - np.clip(x, -theta, theta), atol=1e-15)   # shrinkage identity
        assert np.allclose(orc.soft_threshold(-x, theta), -s, atol=0)      # odd
        assert np.all(s[np.abs(x) <= theta] == 0.0)
        assert np.all(np.abs(s) <= np.abs(x) + 1e-15)
    assert np.array_equal(orc.soft_threshold(x, 0.0), x)
    # prox: argmin_u 1/2 (u-x)^2 + theta |u| by brute force on a fine grid
    grid = np.linspace(-4, 4, 80001)
    for xv in (-2.2, -0.31, 0.0, 0.29, 0.3, 1.7):
        obj = 0.5 * (grid - xv) ** 2 + 0.3 * np.abs(grid)
        assert abs(grid[obj.argmin()] - orc.soft_threshold(np.array([xv]), 0.3)[0]) <= 2e-4


def _lasso_obj(y, M, x, lam):
    return 0.5 * np.sum((y - x @ M.T) ** 2) + lam * np.abs(x).sum()


# P3: the recovery claim (basis-pursuit / RIP paragraph): an exactly k-sparse vector is recovered
# from enough Gaussian measurements; LASSO objective monotone; KKT conditions at convergence
# (these fix theta = mu*lambda, the sign of the gradient step and the transposes).
def test_ista_recovers_k_sparse_and_satisfies_kkt():
    r = _rng(5)
    p, q, k = 32, 64, 3
    M = r.standard_normal((p, q)) / np.sqrt(p)
    x = np.zeros((2, q))
    for row in range(2):
        sup = r.choice(q, k, replace=False)
        x[row, sup] = r.choice([-1.0, 1.0], k) * (1.0 + r.random(k))
    y = x @ M.T
    lam = 5e-3
    S_dec, B_dec, theta, mu = orc.decoder_setup(M, lam)
    assert S_dec.shape == (q, q) and B_dec.shape == (p, q)
    xh, its = orc.ista(y, S_dec, B_dec, theta, 20000, return_iterates=True)
    assert np.array_equal(np.abs(xh) > 1e-3, x != 0)                       # support exact
    assert np.linalg.norm(xh - x) / np.linalg.norm(x) < 1e-2
    objs = [_lasso_obj(y, M, a, lam) for a in its[::50]]
    assert all(b <= a + 1e-12 for a, b in zip(objs, objs[1:]))
    first = [_lasso_obj(y, M, a, lam) for a in its[:40]]
    assert all(b <= a + 1e-12 for a, b in zip(first, first[1:]))
    g = (y - xh @ M.T) @ M                                                # M^T (y - M x^)
    assert np.all(np.abs(g) <= lam * (1 + 1e-6))
    on = xh != 0
    assert np.allclose(g[on], lam * np.sign(xh[on]), rtol=1e-5, atol=1e-9)
    # P11: the iteration map is non-expansive for mu <= 1/L, so steps never grow
    steps = [np.linalg.norm(b - a) for a, b in zip(its[:200], its[1:201])]
    assert all(s2 <= s1 * (1 + 1e-12) + 1e-15 for s1, s2 in zip(steps, steps[1:]))


# step size: L^ is the max absolute row sum of M^T M and bounds its largest eigenvalue.
def test_decoder_setup_step_and_matrices():
    r = _rng(6)
    M = r.standard_normal((5, 5))
    S_dec, B_dec, theta, mu = orc.decoder_setup(M, 0.2)
    G = np.zeros((5, 5))
    for a in range(5):
        for b in range(5):
            G[a, b] = sum(M[k, a] * M[k, b] for k in range(5))
    L = max(sum(abs(G[a, b]) for b in range(5)) for a in range(5))
    assert abs(mu - 1.0 / L) <= 1e-15
    assert L >= np.linalg.eigvalsh(G).max() - 1e-12
    assert np.allclose(S_dec, np.eye(5) - G / L, atol=1e-14)
    assert np.allclose(B_dec, M / L, atol=1e-15)
    assert abs(theta - 0.2 / L) <= 1e-16
    _, _, theta2, mu2 = orc.decoder_setup(M, 0.2, step=0.05)
    assert mu2 == 0.05 and abs(theta2 - 0.01) <= 1e-16


# P4: orthonormal M and mu = 1: one step lands on soft(z M, lambda) and stays there.
def test_orthonormal_sensing_converges_in_one_step():
    r = _rng(7)
    d = 8
    M, _ = np.linalg.qr(r.standard_normal((d, d)))
    z = r.standard_normal((3, d))
    S_dec, B_dec, theta, mu = orc.decoder_setup(M, 0.25, step=1.0)
    a1 = orc.ista(z, S_dec, B_dec, theta, 1)
    a9 = orc.ista(z, S_dec, B_dec, theta, 9)
    expect = np.zeros_like(z)
    for i in range(3):
        for c in range(d):
            v = sum(z[i, k] * M[k, c] for k in range(d))
            expect[i, c] = math.copysign(max(abs(v) - 0.25, 0.0), v)
    assert np.abs(a1 - expect).max() <= 1e-13
    assert np.abs(a9 - expect).max() <= 1e-12


# P5: Phi = I (m = n): default D = I, L^ = 1, so out = soft(Attn, lambda) for every T >= 1; with an
# orthonormal dictionary, out = soft(Attn Psi, lambda) Psi^T.
def test_identity_measurement_with_recovery():
    r = _rng(8)
    n, d = 8, 4
    Q, K, V = r.standard_normal((n, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    attn = brute_attention(Q.tolist(), K.tolist(), V.tolist())
    lam = 0.2
    shr = np.sign(attn) * np.maximum(np.abs(attn) - lam, 0)
    for T in (1, 2, 7):
        out = orc.csat_forward_head(Q, K, V, np.eye(n), T=T, lam=lam)
        assert np.abs(out - shr).max() <= 1e-12
    Psi, _ = np.linalg.qr(r.standard_normal((d, d)))
    w = attn @ Psi
    expect = (np.sign(w) * np.maximum(np.abs(w) - lam, 0)) @ Psi.T
    # G = Psi^T Psi = I up to rounding, L^ = 1 + O(eps): converges geometrically fast
    out = orc.csat_forward_head(Q, K, V, np.eye(n), T=5, lam=lam, Psi=Psi)
    assert np.abs(out - expect).max() <= 1e-10


# P6: lambda = 0 and a well-conditioned D: the iteration is Landweber's and converges to the exact
# inverse, out -> Z D^{-T}, whatever the (invertible) dictionary.  Catches M = Psi D instead of D Psi,
# a missing transpose in B or in the reconstruction, and a wrong sign of the gradient step.
def test_lambda_zero_converges_to_inverse():
    r = _rng(9)
    n, m, d = 12, 6, 5
    Q, K, V = r.standard_normal((4, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    Phi = r.standard_normal((m, n)) / np.sqrt(m)
    D = np.eye(d) + 0.1 * r.standard_normal((d, d))
    Psi, _ = np.linalg.qr(r.standard_normal((d, d)))
    Z = orc.csat_forward_head(Q, K, V, Phi, T=0, lam=0.0)
    expect = np.linalg.solve(D, Z.T).T                                    # rows: z D^{-T}
    for psi in (None, Psi):
        out = orc.csat_forward_head(Q, K, V, Phi, T=3000, lam=0.0, D=D, Psi=psi)
        assert np.abs(out - expect).max() <= 1e-9
    # column-vector statement of the model: z = D Psi alpha, C = Psi alpha
    alpha = np.zeros(d); alpha[[1, 3]] = [2.0, -1.5]
    C = Psi @ alpha
    z = D @ C
    S_dec, B_dec, theta, _ = orc.decoder_setup(D @ Psi, 0.0)
    a = orc.ista(z[None, :], S_dec, B_dec, theta, 3000)
    assert np.abs(orc.reconstruct(a, Psi)[0] - C).max() <= 1e-9


# Default decoder matrix: the leading d x d block of the head's Phi, rows first.
def test_default_decoder_block():
    r = _rng(10)
    n, m, d = 9, 7, 3
    Phi = r.standard_normal((m, n))
    D = orc.default_decoder_matrix(Phi, d)
    for a in range(d):
        for b in range(d):
            assert D[a, b] == Phi[a, b]
    Q, K, V = r.standard_normal((2, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    o1 = orc.csat_forward_head(Q, K, V, Phi, T=4, lam=0.05)
    o2 = orc.csat_forward_head(Q, K, V, Phi, T=4, lam=0.05, D=Phi[:d, :d])
    assert np.array_equal(o1, o2)
    with pytest.raises(AssertionError):
        orc.default_decoder_matrix(Phi[:2], d)


# P7: rows of A~ are probability vectors, so every Z entry lies between the column extremes of V~.
def test_softmax_rows_and_convex_hull():
    r = _rng(11)
    n, m, d = 20, 6, 4
    Q, K, V = 3 * r.standard_normal((5, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    Phi = r.standard_normal((m, n))
    st = {}
    Z = orc.csat_forward_head(Q, K, V, Phi, T=0, lam=0, stages=st)
    A = orc.softmax_rows(orc.compressed_scores(Q, st["Kt"]))
    assert A.shape == (5, m) and np.all(A >= 0) and np.allclose(A.sum(axis=1), 1.0, atol=1e-14)
    assert np.all(Z <= st["Vt"].max(axis=0) + 1e-12) and np.all(Z >= st["Vt"].min(axis=0) - 1e-12)
    # shift invariance and overflow safety of the softmax
    big = orc.softmax_rows(np.array([[1000.0, 1001.0, 999.0]]))
    small = orc.softmax_rows(np.array([[0.0, 1.0, -1.0]]))
    assert np.allclose(big, small, atol=1e-15)
    e = [math.exp(-1), 1.0, math.exp(-2)]
    assert np.allclose(small[0], np.array(e) / sum(e), atol=1e-15)


# P8: linearity of the compression; permutation invariances of Z.
def test_linearity_and_permutation_invariance():
    r = _rng(12)
    n, m, d = 11, 5, 3
    Phi = r.standard_normal((m, n))
    K1, K2 = r.standard_normal((n, d)), r.standard_normal((n, d))
    lhs = orc.compress(Phi, 2.0 * K1 - 0.5 * K2)
    assert np.allclose(lhs, 2.0 * orc.compress(Phi, K1) - 0.5 * orc.compress(Phi, K2), atol=1e-13)
    Q, V = r.standard_normal((4, d)), r.standard_normal((n, d))
    Z = orc.csat_forward_head(Q, K1, V, Phi, T=0, lam=0)
    pt = r.permutation(n)
    Zt = orc.csat_forward_head(Q, K1[pt], V[pt], Phi[:, pt], T=0, lam=0)
    assert np.allclose(Z, Zt, atol=1e-13)
    pm = r.permutation(m)
    Zm = orc.csat_forward_head(Q, K1, V, Phi[pm], T=0, lam=0)
    assert np.allclose(Z, Zm, atol=1e-13)


# The batched driver applies one Phi per head, shared over the batch.
def test_batched_forward_uses_per_head_phi():
    r = _rng(13)
    B, H, n, m, d = 2, 3, 6, 4, 4
    Q, K, V = (r.standard_normal((B, H, n, d)) for _ in range(3))
    Phi = r.standard_normal((H, m, n))
    out = orc.csat_forward(Q, K, V, Phi, T=2, lam=0.05)
    for b in range(B):
        for h in range(H):
            one = orc.csat_forward_head(Q[b, h], K[b, h], V[b, h], Phi[h], T=2, lam=0.05)
            assert np.array_equal(out[b, h], one)


# ----------------------------------------------------------------------------------------
# P9: the measurement-matrix generator
# ----------------------------------------------------------------------------------------
def test_philox_known_answers():
    rows = []
    with open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([int(t, 16) for t in line.split()])
    assert len(rows) == 3
    for w in rows:
        got = phi.philox4x32_10(w[0], w[1], w[2], w[3], w[4], w[5])
        assert [int(x) for x in got] == w[6:10]


def test_phi_layout_counter_and_seed():
    H, m, n, seed = 2, 3, 10, 0x1234567890ABCDEF
    P = phi.phi_gaussian(H, m, n, seed)
    assert P.shape == (H, m, n)
    # element e = (h*m + r)*n + j, block e//4, lane e%4; checked one element at a time
    for (h, r, j) in [(0, 0, 0), (0, 0, 3), (0, 1, 1), (1, 2, 9), (1, 0, 5)]:
        e = (h * m + r) * n + j
        u = [int(x) for x in phi.philox4x32_10(e // 4, 0, 0, 0, seed & 0xFFFFFFFF, seed >> 32)]
        U = [((x >> 9) + 0.5) / 2 ** 23 for x in u]
        g = []
        for a, b in ((0, 1), (2, 3)):
            rad = math.sqrt(-2.0 * math.log(U[a]))
            g += [rad * math.cos(2 * math.pi * U[b]), rad * math.sin(2 * math.pi * U[b])]
        assert abs(P[h, r, j] - g[e % 4] / math.sqrt(m)) <= 1e-15
    assert not np.array_equal(P, phi.phi_gaussian(H, m, n, seed + 1))
    assert np.array_equal(P[1:], phi.phi_gaussian(H, m, n, seed, heads=[1]))


def test_phi_moments_and_normality():
    from scipy import stats
    m, n = 64, 4096
    P = phi.phi_gaussian(1, m, n, 0)[0]
    g = P.ravel() * np.sqrt(m)
    N = g.size
    assert abs(g.mean()) < 4 / np.sqrt(N)
    assert abs(g.var() - 1.0) < 4 * np.sqrt(2 / N)
    assert abs(stats.skew(g)) < 4 * np.sqrt(6 / N)
    assert abs(stats.kurtosis(g)) < 4 * np.sqrt(24 / N)
    assert stats.kstest(g, "norm").pvalue > 1e-3
    cn = (P ** 2).sum(axis=0)                       # squared column norms: mean 1, var 2/m
    assert abs(cn.mean() - 1.0) < 4 * np.sqrt(2 / m / n)
    assert abs(cn.var() - 2 / m) < 0.2 * (2 / m)
    # neighbouring Gaussians of one block and of adjacent blocks are uncorrelated
    for lag in (1, 2, 3, 4):
        c = np.corrcoef(g[:-lag], g[lag:])[0, 1]
        assert abs(c) < 4 / np.sqrt(N)


# ---------------------------------------------------------------------------------------------------
# LISTA recurrence with supplied weights (paper: alpha^{t+1} = eta_theta(S alpha^t + B Z_i), learned S, B, theta)
# ---------------------------------------------------------------------------------------------------
def test_lista_with_ista_weights_is_ista():
    r = np.random.default_rng(21)
    M = r.standard_normal((12, 9)) / 3.0
    Z = r.standard_normal((7, 12))
    S_dec, B_dec, theta, _ = orc.decoder_setup(M, 0.07)
    for T in (1, 2, 9):
        assert np.array_equal(orc.lista(Z, S_dec, B_dec, [theta] * T), orc.ista(Z, S_dec, B_dec, theta, T))


def test_lista_matches_scalar_loops_with_per_layer_thresholds():
    """Brute force: every coordinate by Python loops, non-symmetric S, thresholds that differ per layer."""
    r = np.random.default_rng(22)
    p, q, rows = 3, 4, 2
    S = r.standard_normal((q, q)) * 0.4
    B = r.standard_normal((p, q))
    Z = r.standard_normal((rows, p))
    thetas = [0.3, 0.05, 0.2]
    alpha = [[0.0] * q for _ in range(rows)]
    for th in thetas:
        new = [[0.0] * q for _ in range(rows)]
        for i in range(rows):
            for b in range(q):
                x = sum(alpha[i][a] * S[a][b] for a in range(q)) + sum(Z[i][a] * B[a][b] for a in range(p))
                new[i][b] = (abs(x) - th) * (1 if x > 0 else -1) if abs(x) > th else 0.0
        alpha = new
    assert np.allclose(orc.lista(Z, S, B, thetas), np.array(alpha), rtol=0, atol=1e-14)


def test_lista_special_cases():
    r = np.random.default_rng(23)
    Z = r.standard_normal((5, 6))
    B = r.standard_normal((6, 6))
    # S = 0: every layer forgets the previous iterate, the result is the last layer's shrinkage of Z B
    out = orc.lista(Z, np.zeros((6, 6)), B, [0.5, 0.1, 0.25])
    assert np.array_equal(out, orc.soft_threshold(Z @ B, 0.25))
    # theta = 0, S = I - B (B symmetric positive definite, ||I - B|| < 1): Neumann series, alpha^T -> Z
    A = r.standard_normal((6, 6))
    Bs = 0.5 * np.eye(6) + 0.05 * (A @ A.T) / 6
    out = orc.lista(Z, np.eye(6) - Bs, Bs, [0.0] * 400)
    assert np.allclose(out, Z, atol=1e-9)
    # transposed S must give a different answer (row-vector convention alpha S)
    Sn = r.standard_normal((6, 6)) * 0.3
    assert not np.allclose(orc.lista(Z, Sn, B, [0.1] * 3), orc.lista(Z, Sn.T, B, [0.1] * 3))


def test_lista_per_layer_weights_match_scalar_loops():
    """Brute force with a different S_t, B_t and theta_t in every layer."""
    r = np.random.default_rng(24)
    p, q, rows, T = 3, 4, 2, 3
    S = r.standard_normal((T, q, q)) * 0.4
    B = r.standard_normal((T, p, q))
    Z = r.standard_normal((rows, p))
    thetas = [0.25, 0.02, 0.15]
    alpha = [[0.0] * q for _ in range(rows)]
    for t in range(T):
        new = [[0.0] * q for _ in range(rows)]
        for i in range(rows):
            for b in range(q):
                x = sum(alpha[i][a] * S[t][a][b] for a in range(q)) + sum(Z[i][a] * B[t][a][b] for a in range(p))
                new[i][b] = (abs(x) - thetas[t]) * (1 if x > 0 else -1) if abs(x) > thetas[t] else 0.0
        alpha = new
    assert np.allclose(orc.lista(Z, S, B, thetas), np.array(alpha), rtol=0, atol=1e-14)


def test_lista_per_layer_weights_closed_forms():
    r = np.random.default_rng(25)
    T, q = 4, 5
    Z = r.standard_normal((6, q))
    S = r.standard_normal((T, q, q)) * 0.5
    B = r.standard_normal((T, q, q))
    # theta = 0: the recurrence is linear, alpha^T = sum_t Z B_t S_{t+1} S_{t+2} ... S_{T-1}
    want = np.zeros((6, q))
    for t in range(T):
        term = Z @ B[t]
        for u in range(t + 1, T):
            term = term @ S[u]
        want += term
    assert np.allclose(orc.lista(Z, S, B, [0.0] * T), want, rtol=0, atol=1e-12)
    # the layers do not commute: the reversed stack gives something else
    assert not np.allclose(orc.lista(Z, S[::-1], B[::-1], [0.0] * T), want)
    # S_t = 0 in the last layer: only that layer's B and threshold count
    S0 = S.copy()
    S0[-1] = 0.0
    assert np.array_equal(orc.lista(Z, S0, B, [0.3, 0.2, 0.1, 0.05]), orc.soft_threshold(Z @ B[-1], 0.05))
    # the same matrix in every layer is the shared form
    th = [0.2, 0.1, 0.3, 0.05]
    tied = orc.lista(Z, S[1], B[2], th)
    assert np.array_equal(orc.lista(Z, np.stack([S[1]] * T), np.stack([B[2]] * T), th), tied)
    # one S, one B and one threshold per layer, or an error
    for bad in [(S[:3], B, th), (S, B[:3], th), (S, B, th[:3]), (S, B[0], th)]:
        try:
            orc.lista(Z, *bad)
        except ValueError:
            continue
        raise AssertionError("inconsistent per-layer weights accepted")


def test_forward_with_per_layer_weights_uses_them():
    """The whole forward hands layer t of head h its own matrices: equal to the stages composed by hand."""
    r = np.random.default_rng(26)
    Bt, H, n, nq, d, m, T = 2, 2, 12, 5, 4, 6, 3
    Q, K, V = (r.standard_normal((Bt, H, s, d)) for s in (nq, n, n))
    Phi = r.standard_normal((H, m, n)) / np.sqrt(m)
    S = r.standard_normal((T, H, d, d)) * 0.4
    Bm = r.standard_normal((T, H, d, d)) * 0.6
    th = np.abs(r.standard_normal((T, H))) * 0.05
    Psi = r.standard_normal((d, d))
    out = orc.csat_forward(Q, K, V, Phi, T=T, lam=0.0, Psi=Psi, weights=(S, Bm, list(th)))
    for b in range(Bt):
        for h in range(H):
            Z = orc.csat_forward_head(Q[b, h], K[b, h], V[b, h], Phi[h], T=0, lam=0.0)
            a = np.zeros((nq, d))
            for t in range(T):
                a = orc.soft_threshold(a @ S[t, h] + Z @ Bm[t, h], th[t, h])
            assert np.allclose(out[b, h], a @ Psi.T, rtol=0, atol=1e-13)


def test_forward_with_supplied_weights_uses_them():
    w = wl.shrink(wl.CONFIGS["c1"], n=32, n_q=8, m=16, d=8)
    inp = wl.make_inputs(w)
    Phi = phi.phi_gaussian(1, w.m, w.n, 0)
    r = np.random.default_rng(24)
    S = r.standard_normal((1, 8, 8)) * 0.2
    B = r.standard_normal((1, 8, 8)) * 0.5
    thetas = [[0.05], [0.02]]
    st = []
    out = orc.csat_forward(inp["Q"], inp["K"], inp["V"], Phi, T=2, lam=123.0, weights=(S, B, thetas), stages=st)
    Z = st[0]["Z"]
    a1 = orc.soft_threshold(Z @ B[0], 0.05)
    a2 = orc.soft_threshold(a1 @ S[0] + Z @ B[0], 0.02)
    assert np.allclose(out[0, 0], a2, atol=1e-14)


# ---------------------------------------------------------------------------------------------------
# Rademacher measurement matrices (the second of the three ensembles the paper lists)
# ---------------------------------------------------------------------------------------------------
def _philox_scalar(ctr, key):
    """Philox4x32-10 on Python ints, written from the published round function (checked against the
    known-answer vectors below before it is used)."""
    c = list(ctr)
    k0, k1 = key
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k0, p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k1, p0 & 0xFFFFFFFF]
        k0, k1 = (k0 + 0x9E3779B9) & 0xFFFFFFFF, (k1 + 0xBB67AE85) & 0xFFFFFFFF
    return c


def test_rademacher_layout_by_scalar_brute_force():
    # the scalar routine reproduces the published known-answer vectors
    assert _philox_scalar([0, 0, 0, 0], [0, 0]) == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]
    assert _philox_scalar([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2) == [0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD]
    H, m, n, seed = 2, 5, 77, 0x0123456789ABCDEF
    got = phi.phi_rademacher(H, m, n, seed)
    for (h, r, j) in [(0, 0, 0), (0, 0, 31), (0, 0, 32), (0, 1, 50), (0, 4, 76), (1, 0, 0), (1, 3, 5), (1, 4, 76)]:
        e = (h * m + r) * n + j
        q = e // 128
        words = _philox_scalar([q & 0xFFFFFFFF, q >> 32, 1, 0], [seed & 0xFFFFFFFF, seed >> 32])
        bit = (words[(e // 32) % 4] >> (e % 32)) & 1
        assert got[h, r, j] == (-1.0 if bit else 1.0) / math.sqrt(m)


def test_rademacher_is_a_sign_matrix_with_unit_columns():
    H, m, n = 3, 64, 500
    P = phi.phi_rademacher(H, m, n, 7)
    assert np.array_equal(np.abs(P), np.full_like(P, 1.0 / 8.0))
    assert np.allclose((P ** 2).sum(axis=1), 1.0, atol=1e-15)                 # every column has norm exactly 1
    assert abs(P.mean()) * 8.0 < 4.0 / math.sqrt(P.size)                      # balanced signs (4 sigma)
    # rows are nearly orthogonal: off-diagonal Gram entries are sums of n independent signs / m
    G = P[0] @ P[0].T
    off = G[~np.eye(m, dtype=bool)]
    assert np.abs(off).max() < 5.0 * math.sqrt(n) / m and abs(off.mean()) < 5.0 * math.sqrt(n) / m / math.sqrt(off.size) * 2
    # another seed, another head: different matrices
    assert not np.array_equal(P[0], P[1])
    assert not np.array_equal(P, phi.phi_rademacher(H, m, n, 8))
    # and not the Gaussian ensemble's sign pattern
    assert not np.array_equal(np.sign(P), np.sign(phi.phi_gaussian(H, m, n, 7)))


# ---------------------------------------------------------------------------------------------------
# Structured Hadamard measurement matrices
# ---------------------------------------------------------------------------------------------------
def test_hadamard_ensemble_against_the_library_hadamard_matrix():
    from scipy.linalg import hadamard
    H, m, n, seed = 2, 24, 64, 11
    P = phi.phi_hadamard(H, m, n, seed)
    N, rows = phi.hadamard_rows(H, m, n, seed)
    assert N == 64 and all(len(set(rows[h])) == m for h in range(H))      # distinct rows
    W = hadamard(N).astype(np.float64)
    for h in range(H):
        signs = P[h, 0] * math.sqrt(m) * W[rows[h, 0]]                     # recovers the column signs from row 0
        assert np.array_equal(np.abs(signs), np.ones(n))
        assert np.array_equal(P[h], W[rows[h]] * signs[None, :] / math.sqrt(m))
        assert np.allclose(P[h] @ P[h].T, np.eye(m) * n / m, atol=1e-12)  # orthogonal rows when n is a power of two
        assert abs(signs.sum()) < n                                        # not all the same sign
    assert not np.array_equal(rows[0], rows[1])
    # truncated columns (n not a power of two): still a sign matrix with unit columns, rows of the 256 x 256 matrix
    P = phi.phi_hadamard(1, 16, 197, 3)
    N, rows = phi.hadamard_rows(1, 16, 197, 3)
    assert N == 256 and np.array_equal(np.abs(P), np.full_like(P, 0.25))
    W = hadamard(256).astype(np.float64)
    G = (P[0] * 4.0) * W[rows[0]][:, :197]                                 # = column signs in every row
    assert np.array_equal(G, np.tile(G[:1], (16, 1)))


# ---------------------------------------------------------------------------------------------------
# Separate measurement matrices for keys and values (paper: K~ = Phi_K K, V~ = Phi_V V)
# ---------------------------------------------------------------------------------------------------
def test_separate_value_matrix():
    w = wl.shrink(wl.CONFIGS["c1"], n=40, n_q=6, m=12, d=8)
    inp = wl.make_inputs(w)
    both = phi.phi_gaussian(2, w.m, w.n, 5)
    Pk, Pv = both[:1], both[1:]
    # the same matrix passed twice is the shared-matrix forward
    a = orc.csat_forward(inp["Q"], inp["K"], inp["V"], Pk, T=3, lam=0.01)
    b = orc.csat_forward(inp["Q"], inp["K"], inp["V"], Pk, T=3, lam=0.01, Phi_V=Pk)
    assert np.array_equal(a, b)
    # different matrices: scores from Phi_K K, values from Phi_V V, by hand
    st = []
    out = orc.csat_forward(inp["Q"], inp["K"], inp["V"], Pk, T=0, lam=0.0, Phi_V=Pv, stages=st)
    Q, K, V = (inp[k][0, 0].astype(np.float64) for k in "QKV")
    S = Q @ (Pk[0] @ K).T / math.sqrt(w.d)
    A = np.exp(S - S.max(axis=1, keepdims=True)); A /= A.sum(axis=1, keepdims=True)
    assert np.allclose(out[0, 0], A @ (Pv[0] @ V), atol=1e-13)
    assert not np.allclose(out, orc.csat_forward(inp["Q"], inp["K"], inp["V"], Pv, T=0, lam=0.0, Phi_V=Pk))
    # the decoder's default matrix is the block of Phi_V
    st = []
    orc.csat_forward(inp["Q"], inp["K"], inp["V"], Pk, T=2, lam=0.01, Phi_V=Pv, stages=st)
    S_ref, B_ref, th_ref, mu_ref = orc.decoder_setup(Pv[0][:w.d, :w.d], 0.01)
    assert np.array_equal(st[0]["B_dec"], B_ref) and st[0]["theta"] == th_ref


# ---------------------------------------------------------------------------------------------------
# input projections (paper: Q = X W^Q, K = X W^K, V = X W^V)
# ---------------------------------------------------------------------------------------------------
def test_project_qkv_matches_scalar_loops_and_layout():
    r = np.random.default_rng(61)
    B, n, dm, H, d = 2, 3, 5, 2, 4
    X = r.standard_normal((B, n, dm))
    W = r.standard_normal((dm, 3 * H * d))
    Q, K, V = orc.project_qkv(X, W, H, d)
    for which, P in enumerate((Q, K, V)):
        assert P.shape == (B, H, n, d)
        for b in range(B):
            for h in range(H):
                for i in range(n):
                    for c in range(d):
                        want = sum(X[b][i][k] * W[k][(which * H + h) * d + c] for k in range(dm))
                        assert abs(P[b, h, i, c] - want) < 1e-13
    # closed forms: a one-hot token picks a row of W; an identity-like W copies X into the heads
    E = np.zeros((1, 1, dm)); E[0, 0, 3] = 1.0
    Q1, K1, V1 = orc.project_qkv(E, W, H, d)
    assert np.array_equal(Q1[0, :, 0, :].reshape(-1), W[3, :H * d])
    assert np.array_equal(K1[0, :, 0, :].reshape(-1), W[3, H * d:2 * H * d])
    assert np.array_equal(V1[0, :, 0, :].reshape(-1), W[3, 2 * H * d:])
    Wi = np.zeros((H * d, 3 * H * d)); Wi[:, :H * d] = np.eye(H * d); Wi[:, H * d:2 * H * d] = 2 * np.eye(H * d)
    Xi = r.standard_normal((B, n, H * d))
    Q2, K2, V2 = orc.project_qkv(Xi, Wi, H, d)
    assert np.array_equal(Q2.transpose(0, 2, 1, 3).reshape(B, n, H * d), Xi)
    assert np.array_equal(K2.transpose(0, 2, 1, 3).reshape(B, n, H * d), 2 * Xi)
    assert not V2.any()


# ---------------------------------------------------------------------------------------------------
# backward (vector-Jacobian product of the forward with respect to Q, K, V)
# ---------------------------------------------------------------------------------------------------
def _torch_forward(Q, K, V, Phi, Phi_v, S_l, B_l, thetas, Psi, scale, forced_masks=None):
    """The forward written with torch float64 ops, for autograd (an independent derivation of the gradient).
    forced_masks [T,n_q,d]: layer t computes masks[t] o (x - theta sign(x)) instead of the shrinkage, i.e. the
    shrinkage with its decisions |x| > theta taken from outside."""
    import torch
    Kt, Vt = Phi @ K, Phi_v @ V
    A = torch.softmax(scale * (Q @ Kt.T), dim=1)
    Z = A @ Vt
    alpha = torch.zeros_like(Z)
    out = Z
    for t, (S_t, B_t, th) in enumerate(zip(S_l, B_l, thetas)):
        x = alpha @ S_t + Z @ B_t
        if forced_masks is None:
            alpha = torch.sign(x) * torch.relu(torch.abs(x) - th)
        else:
            alpha = forced_masks[t] * (x - th * torch.sign(x))
        out = alpha
    if Psi is not None and len(thetas) > 0:
        out = out @ Psi.T
    return out


def _backward_case(seed, T, with_psi, separate, untied):
    import torch
    r = np.random.default_rng(seed)
    n, nq, d, m = 14, 6, 5, 7
    Q, K, V = r.standard_normal((nq, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    Phi = r.standard_normal((m, n)) / np.sqrt(m)
    Phi_v = r.standard_normal((m, n)) / np.sqrt(m) if separate else None
    Psi = (np.eye(d) + 0.3 * r.standard_normal((d, d))) if with_psi else None
    G = r.standard_normal((nq, d))
    lam = 0.15
    if untied:
        S = 0.5 * np.eye(d) + 0.2 * r.standard_normal((T, d, d))
        Bm = 0.5 * r.standard_normal((T, d, d))
        thetas = list(0.02 + 0.05 * r.random(T))
        weights = (S, Bm, thetas)
        S_l, B_l = list(S), list(Bm)
    else:
        weights = None
        Dm = orc.default_decoder_matrix(Phi if Phi_v is None else Phi_v, d)
        M = Dm if Psi is None else Dm @ Psi
        S_dec, B_dec, theta, _ = orc.decoder_setup(M, lam)
        S_l, B_l, thetas = [S_dec] * T, [B_dec] * T, [float(theta)] * T
    st = {}
    got = orc.csat_backward_head(Q, K, V, Phi, G, T=T, lam=lam, Psi=Psi, weights=weights, Phi_v_h=Phi_v, stages=st)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    t = lambda x: None if x is None else torch.tensor(x, dtype=torch.float64)
    # one leaf per layer for every decoder parameter, so that autograd gives the per-layer gradients
    tS = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in S_l]
    tB = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in B_l]
    tth = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in thetas]
    tPsi = None if Psi is None else torch.tensor(Psi, dtype=torch.float64, requires_grad=True)
    # the measurement matrices as leaves too (the decoder's matrices above are constants for autograd, i.e. held fixed)
    tPhi = torch.tensor(Phi, dtype=torch.float64, requires_grad=True)
    tPhiv = tPhi if Phi_v is None else torch.tensor(Phi_v, dtype=torch.float64, requires_grad=True)
    out = _torch_forward(tq, tk, tv, tPhi, tPhiv, tS, tB, tth, tPsi, 1.0 / np.sqrt(d))
    # the torch forward is the oracle's forward
    ref_out = orc.csat_forward_head(Q, K, V, Phi, T=T, lam=lam, Psi=Psi, weights=weights, Phi_v_h=Phi_v)
    assert np.allclose(out.detach().numpy(), ref_out, rtol=0, atol=1e-12)
    (out * t(G)).sum().backward()
    for name, g, ref in zip("QKV", got, (tq.grad, tk.grad, tv.grad)):
        assert np.allclose(g, ref.numpy(), rtol=1e-10, atol=1e-12), (name, seed, T)
    # gradients with respect to the decoder's parameters, layer by layer
    assert st["dS"].shape == (T, d, d) and st["dB"].shape == (T, d, d) and st["dtheta"].shape == (T,)
    for l in range(T):
        gS = tS[l].grad.numpy() if tS[l].grad is not None else np.zeros((d, d))     # layer 0 multiplies alpha^0 = 0
        assert np.allclose(st["dS"][l], gS, rtol=1e-10, atol=1e-12), ("dS", seed, l)
        assert np.allclose(st["dB"][l], tB[l].grad.numpy(), rtol=1e-10, atol=1e-12), ("dB", seed, l)
        assert np.allclose(st["dtheta"][l], tth[l].grad.numpy(), rtol=1e-10, atol=1e-12), ("dtheta", seed, l)
    if Psi is not None and T > 0:
        assert np.allclose(st["dPsi"], tPsi.grad.numpy(), rtol=1e-10, atol=1e-12), ("dPsi", seed)
    if Phi_v is None:
        assert np.allclose(st["dPhi_K"] + st["dPhi_V"], tPhi.grad.numpy(), rtol=1e-10, atol=1e-12), ("dPhi", seed)
    else:
        assert np.allclose(st["dPhi_K"], tPhi.grad.numpy(), rtol=1e-10, atol=1e-12), ("dPhi_K", seed)
        assert np.allclose(st["dPhi_V"], tPhiv.grad.numpy(), rtol=1e-10, atol=1e-12), ("dPhi_V", seed)
    if T > 0:
        assert st["masks"].shape == (T, nq, d) and st["xs"].shape == (T, nq, d)
        assert np.array_equal(st["masks"], np.abs(st["xs"]) > np.asarray(thetas)[:, None, None])
    return Q, K, V, Phi, Phi_v, Psi, G, lam, weights, got, st


def test_backward_with_supplied_shrinkage_decisions():
    """masks= replaces the oracle's own decisions |x_t| > theta_t.  Pinned by autograd through a forward whose
    layers compute masks[t] o (x - theta sign(x)) with RANDOM masks (so that layer, row and column indices all
    matter); the gradients with respect to Q, K, V depend on the masks and on constant matrices only, so they must
    agree exactly.  The oracle's own masks passed back in change nothing."""
    import torch
    for seed, T, with_psi, separate, untied in [(91, 3, False, False, False), (92, 4, True, True, True)]:
        Q, K, V, Phi, Phi_v, Psi, G, lam, weights, got, st = _backward_case(seed, T, with_psi, separate, untied)
        kw = dict(T=T, lam=lam, Psi=Psi, weights=weights, Phi_v_h=Phi_v)
        same = orc.csat_backward_head(Q, K, V, Phi, G, masks=st["masks"], **kw)
        for a, b in zip(got, same):
            assert np.array_equal(a, b)
        r = np.random.default_rng(seed + 100)
        forced = r.random(st["masks"].shape) < 0.6
        assert (forced != st["masks"]).any() and len({forced[l].tobytes() for l in range(T)}) == T
        d = Q.shape[1]
        if weights is None:
            Dm = orc.default_decoder_matrix(Phi if Phi_v is None else Phi_v, d)
            S_dec, B_dec, theta, _ = orc.decoder_setup(Dm if Psi is None else Dm @ Psi, lam)
            S_l, B_l, thetas = [S_dec] * T, [B_dec] * T, [float(theta)] * T
        else:
            S_l, B_l, thetas = list(weights[0]), list(weights[1]), list(weights[2])
        t = lambda x: None if x is None else torch.tensor(x, dtype=torch.float64)
        tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
        out = _torch_forward(tq, tk, tv, t(Phi), t(Phi if Phi_v is None else Phi_v), [t(x) for x in S_l],
                             [t(x) for x in B_l], thetas, t(Psi), 1.0 / np.sqrt(d),
                             forced_masks=torch.tensor(forced, dtype=torch.float64))
        (out * t(G)).sum().backward()
        with_forced = orc.csat_backward_head(Q, K, V, Phi, G, masks=forced, **kw)
        for name, g, ref in zip("QKV", with_forced, (tq.grad, tk.grad, tv.grad)):
            assert np.allclose(g, ref.numpy(), rtol=1e-10, atol=1e-12), (name, seed)
        # whole-batch wrapper hands every (batch, head) its own masks
        Qb, Kb, Vb, Gb = (np.stack([x, x[::-1]])[None] for x in (Q, K, V, G))          # B = 1, H = 2
        Phib = np.stack([Phi, Phi])
        wb = None if weights is None else (np.stack([weights[0]] * 2, axis=1), np.stack([weights[1]] * 2, axis=1),
                                           [[th, th] for th in weights[2]])
        mb = np.stack([forced, st["masks"][:, ::-1]])[None]
        full = orc.csat_backward(Qb, Kb, Vb, Phib, Gb, T=T, lam=lam, Psi=Psi, weights=wb,
                                 Phi_V=None if Phi_v is None else np.stack([Phi_v, Phi_v]), masks=mb)
        for x, y in zip(full, with_forced):
            assert np.array_equal(x[0, 0], y)


def test_backward_matches_autograd():
    for seed, T, with_psi, separate, untied in [(81, 0, False, False, False), (82, 1, False, False, False),
                                                (83, 4, True, False, False), (84, 3, False, True, False),
                                                (85, 5, True, True, True), (86, 2, False, False, True)]:
        _backward_case(seed, T, with_psi, separate, untied)


def test_backward_matches_central_differences():
    """dL/dx_k by (L(x + h e_k) - L(x - h e_k)) / 2h with L = sum(out o G), along random directions, on a case
    whose iterates keep clear of the kinks of eta by far more than the step."""
    Q, K, V, Phi, Phi_v, Psi, G, lam, weights, got, st = _backward_case(87, 4, True, False, False)
    assert st["min_margin"].min() > 1e-4
    r = np.random.default_rng(88)
    L = lambda q, k, v: float((orc.csat_forward_head(q, k, v, Phi, T=4, lam=lam, Psi=Psi, weights=weights) * G).sum())
    h = 1e-6
    for which in range(3):
        for _ in range(4):
            dirs = [np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)]
            dirs[which] = r.standard_normal(dirs[which].shape)
            fd = (L(Q + h * dirs[0], K + h * dirs[1], V + h * dirs[2]) - L(Q - h * dirs[0], K - h * dirs[1], V - h * dirs[2])) / (2 * h)
            an = float((got[which] * dirs[which]).sum())
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (which, fd, an)


def test_backward_special_cases():
    r = np.random.default_rng(89)
    n, nq, d, m = 9, 4, 3, 5
    Q, K, V = r.standard_normal((nq, d)), r.standard_normal((n, d)), r.standard_normal((n, d))
    Phi = r.standard_normal((m, n))
    G = r.standard_normal((nq, d))
    # T = 0 and m = 1: the softmax over one measurement is 1, out = Phi V for every query: dQ = 0, dK = 0,
    # dV = Phi^T (sum of the rows of G)
    dQ, dK, dV = orc.csat_backward_head(Q, K, V, Phi[:1], G, T=0, lam=0.0)
    assert np.allclose(dQ, 0, atol=1e-15) and np.allclose(dK, 0, atol=1e-15)
    assert np.allclose(dV, Phi[:1].T @ G.sum(axis=0, keepdims=True), rtol=1e-12, atol=1e-14)
    # a threshold above every |x|: the output is 0 and so is every gradient
    big = (np.zeros((d, d)), np.eye(d), [1e6, 1e6])
    for g in orc.csat_backward_head(Q, K, V, Phi, G, T=2, lam=0.0, weights=big):
        assert not g.any()
    # theta = 0, S = 0, B = I, one layer: the decoder is the identity, the gradient is the T = 0 gradient
    ident = (np.zeros((d, d)), np.eye(d), [0.0])
    a = orc.csat_backward_head(Q, K, V, Phi, G, T=1, lam=0.0, weights=ident)
    b = orc.csat_backward_head(Q, K, V, Phi, G, T=0, lam=0.0)
    for x, y in zip(a, b):
        assert np.allclose(x, y, rtol=1e-12, atol=1e-14)
    # whole-batch wrapper = the heads one by one
    Qb, Kb, Vb = (r.standard_normal((2, 2, s, d)) for s in (nq, n, n))
    Phib = r.standard_normal((2, m, n))
    Gb = r.standard_normal((2, 2, nq, d))
    full = orc.csat_backward(Qb, Kb, Vb, Phib, Gb, T=2, lam=0.1)
    one = orc.csat_backward_head(Qb[1, 0], Kb[1, 0], Vb[1, 0], Phib[0], Gb[1, 0], T=2, lam=0.1)
    for x, y in zip(full, one):
        assert np.array_equal(x[1, 0], y)
