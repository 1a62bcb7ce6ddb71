"""Pins the float64 checker to what the paper and the mathematics fix (no GPU)."""
import math

import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc


def tiny(widths=(5, 4, 3, 2), l=12, nS=7, C=1.5, seed=7, x="uniform", n_vec=2):
    return wl.make_custom(widths, l, nS, C, seed, x=x, n_vec=n_vec)


# ------------------------------------------------------------------ layout (Section 2.1)
def test_theta_layout_is_column_concatenation():
    widths = [3, 2, 2]
    n = orc.num_params(widths)
    assert n == 3 * 2 + 2 + 2 * 2 + 2 == wl.num_params(widths)
    theta = np.arange(1, n + 1, dtype=np.float64)
    (W1, b1), (W2, b2) = orc.unpack(theta, widths)
    # w^1 = [w_11 w_21 w_31 w_12 w_22 w_32]: column 1 of W^1 first
    assert W1[:, 0].tolist() == [1, 2, 3] and W1[:, 1].tolist() == [4, 5, 6]
    assert b1.tolist() == [7, 8]
    assert W2[:, 0].tolist() == [9, 10] and W2[:, 1].tolist() == [11, 12]
    assert b2.tolist() == [13, 14]
    assert np.array_equal(orc.pack([(W1, b1), (W2, b2)]), theta)
    assert [(s.start, s.stop) for s in orc.block_slices(widths)] == [(0, 8), (8, 14)]
    assert [(a, c) for a, _, c in wl.layer_offsets(widths)] == [(0, 8), (8, 14)]


# ------------------------------------------------------------------ f (Eq. obj-function)
def test_f_at_zero_is_one_for_one_hot_labels():
    p = tiny()
    theta0 = np.zeros(p["n"])
    # hidden z = 1/2, output z^L = b^L = 0, so every row contributes ||y||^2 = 1
    assert orc.fun(theta0, p["widths"], p["C"], p["X"], p["Y"]) == pytest.approx(1.0, abs=1e-15)
    Z = orc.forward(theta0, p["widths"], p["X"])
    assert np.all(Z[1] == 0.5) and np.all(Z[2] == 0.5) and np.all(Z[3] == 0.0)


def test_hand_computed_2_1_1_network():
    # x = (1, -2); W^1 = [[0.5],[0.25]], b^1 = 0.1; W^2 = [[-3]], b^2 = 0.7; y = 1; C = 4
    widths = [2, 1, 1]
    theta = np.array([0.5, 0.25, 0.1, -3.0, 0.7])
    x = np.array([[1.0, -2.0]])
    y = np.array([[1.0]])
    s1 = 0.5 * 1.0 + 0.25 * (-2.0) + 0.1          # = 0.1
    z1 = 1.0 / (1.0 + math.exp(-s1))
    z2 = -3.0 * z1 + 0.7
    reg = (0.25 + 0.0625 + 0.01 + 9.0 + 0.49) / (2 * 4.0)
    assert orc.fun(theta, widths, 4.0, x, y) == pytest.approx(reg + (z2 - 1.0) ** 2, rel=1e-14)
    # gradient by the chain rule, written out by hand
    e = 2.0 * (z2 - 1.0)
    dz1 = e * (-3.0) * z1 * (1 - z1)
    expect = np.array([dz1 * 1.0, dz1 * -2.0, dz1, e * z1, e]) + theta / 4.0
    assert np.allclose(orc.grad(theta, widths, 4.0, x, y), expect, rtol=1e-13, atol=0)
    # Jacobian of the single output
    J = orc.jacobian(theta, widths, x[0])
    dj = -3.0 * z1 * (1 - z1)
    assert np.allclose(J, [[dj * 1.0, dj * -2.0, dj, z1, 1.0]], rtol=1e-13, atol=0)


def test_regulariser_includes_biases():
    p = tiny()
    th = p["theta"].astype(np.float64)
    sl = orc.block_slices(p["widths"])[0]
    a, b = p["widths"][0], p["widths"][1]
    bias_pos = sl.start + a * b            # first bias of layer 1
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    th2 = th.copy()
    th2[bias_pos] += 1.0
    # the 1/C part of d f / d b changes by exactly 1/C in the L2 term's derivative
    f_reg = lambda t: t @ t / (2 * p["C"])
    assert f_reg(th2) - f_reg(th) == pytest.approx((2 * th[bias_pos] + 1) / (2 * p["C"]))
    G = orc.gauss_newton_dense(th, p["widths"], 1e300, p["X"][p["idx"]])  # no I/C
    G2 = orc.gauss_newton_dense(th, p["widths"], p["C"], p["X"][p["idx"]])
    assert np.allclose(np.diag(G2 - G), 1.0 / p["C"])        # identity on all n coordinates
    assert g.shape == th.shape


# ------------------------------------------------------------------ gradient (Eq. whole-gradient)
def fd_grad(fn, th, h=1e-5):
    out = np.zeros_like(th)
    for k in range(th.size):
        e = np.zeros_like(th)
        e[k] = h
        out[k] = (fn(th + e) - fn(th - e)) / (2 * h)
    return out


@pytest.mark.parametrize("widths", [(5, 4, 3, 2), (4, 3), (3, 5, 1), (2, 3, 3, 3, 2)])
def test_gradient_matches_finite_differences(widths):
    p = tiny(widths=widths, seed=11)
    th = p["theta"].astype(np.float64)
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    fd = fd_grad(lambda t: orc.fun(t, p["widths"], p["C"], p["X"], p["Y"]), th)
    assert np.linalg.norm(g - fd) <= 1e-7 * np.linalg.norm(fd)


def test_gradient_at_zero_closed_form():
    # theta = 0: only b^L has a non-zero derivative through the loss: (1/l) sum 2 (0 - y)
    p = tiny()
    g = orc.grad(np.zeros(p["n"]), p["widths"], p["C"], p["X"], p["Y"])
    sl = orc.block_slices(p["widths"])[-1]
    a, b = p["widths"][-2], p["widths"][-1]
    gbL = g[sl][a * b:]
    assert np.allclose(gbL, -2.0 * p["Y"].mean(axis=0))
    gWL = g[sl][:a * b].reshape(b, a)                    # row j = column j of W^L
    assert np.allclose(gWL, (-2.0 * p["Y"].mean(axis=0))[:, None] * 0.5)
    assert np.all(g[: sl.start] == 0.0)                  # W^L = 0 blocks everything below


# ------------------------------------------------------------------ Jacobian (Eq. jacobian, Section 3.3)
@pytest.mark.parametrize("widths", [(5, 4, 3, 2), (4, 3), (3, 5, 1), (2, 3, 3, 3, 2)])
def test_jacobian_matches_finite_differences_of_the_output(widths):
    p = tiny(widths=widths, seed=5)
    th = p["theta"].astype(np.float64)
    x = p["X"][3]
    J = orc.jacobian(th, p["widths"], x)
    h = 1e-6
    for k in range(th.size):
        e = np.zeros_like(th)
        e[k] = h
        col = (orc.forward(th + e, p["widths"], x[None])[-1][0]
               - orc.forward(th - e, p["widths"], x[None])[-1][0]) / (2 * h)
        assert np.allclose(J[:, k], col, rtol=1e-6, atol=1e-9)


def test_jacobian_output_bias_columns_are_identity():
    p = tiny()
    J = orc.jacobian(p["theta"], p["widths"], p["X"][0])
    nL = p["widths"][-1]
    assert np.array_equal(J[:, -nL:], np.eye(nL))        # Eq. (xtow-jaco-bias), m = L
    # and the w^L columns are z^{L-1}_t on the matching output, zero elsewhere (Eq. xtow-jaco)
    z = orc.forward(p["theta"], p["widths"], p["X"][:1])[-2][0]
    a = p["widths"][-2]
    sl = orc.block_slices(p["widths"])[-1]
    for j in range(nL):
        blockcols = J[:, sl.start + j * a: sl.start + (j + 1) * a]
        expect = np.zeros_like(blockcols)
        expect[j] = z
        assert np.allclose(blockcols, expect, rtol=1e-15)


# ------------------------------------------------------------------ G (Eq. def-gauss-newton / sampled-Gauss)
def test_G_symmetric_and_positive_definite():
    p = tiny()
    XS = p["X"][p["idx"]]
    u, v = p["vs"][0].astype(np.float64), p["vs"][1].astype(np.float64)
    Gu = orc.Gv(p["theta"], p["widths"], p["C"], XS, u)
    Gv_ = orc.Gv(p["theta"], p["widths"], p["C"], XS, v)
    assert u @ Gv_ == pytest.approx(v @ Gu, rel=1e-12)
    assert v @ Gv_ >= v @ v / p["C"]
    G = orc.gauss_newton_dense(p["theta"], p["widths"], p["C"], XS)
    assert np.allclose(G, G.T, rtol=0, atol=1e-14)
    assert np.linalg.eigvalsh(G).min() >= 1.0 / p["C"] - 1e-12


def test_G_linear_in_v():
    p = tiny()
    XS = p["X"][p["idx"]]
    u, v = p["vs"][0].astype(np.float64), p["vs"][1].astype(np.float64)
    f = lambda w: orc.Gv(p["theta"], p["widths"], p["C"], XS, w)
    assert np.allclose(f(2.5 * u - 0.5 * v), 2.5 * f(u) - 0.5 * f(v), rtol=1e-12, atol=1e-13)


def test_no_hidden_layer_closed_form_scalar_output():
    # L = 1, n_L = 1, linear output: J^i = [x^T, 1], so G = I/C + (2/|S|) Xt^T Xt
    p = wl.make_custom([6, 1], 20, 9, 0.7, seed=3, x="normal", n_vec=1)
    XS = p["X"][p["idx"]].astype(np.float64)
    Xt = np.hstack([XS, np.ones((len(XS), 1))])
    G = np.eye(7) / p["C"] + 2.0 / len(XS) * Xt.T @ Xt
    v = p["v"].astype(np.float64)
    assert np.allclose(orc.Gv(p["theta"], p["widths"], p["C"], XS, v), G @ v, rtol=1e-13)
    assert np.allclose(orc.Gv_definition(p["theta"], p["widths"], p["C"], XS, v), G @ v, rtol=1e-13)
    assert np.allclose(orc.gauss_newton_dense(p["theta"], p["widths"], p["C"], XS), G, rtol=1e-13)
    # one block only: the block-diagonal matrix is G itself
    assert np.allclose(orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, v), G @ v, rtol=1e-13)


def test_no_hidden_layer_closed_form_vector_output():
    # L = 1, n_L = K: G = I/C + (2/|S|) I_K (x) Xt^T Xt in theta's (w_1..w_K, b) order
    K, n0 = 3, 4
    p = wl.make_custom([n0, K], 15, 8, 2.0, seed=4, x="normal", n_vec=1)
    XS = p["X"][p["idx"]].astype(np.float64)
    Xt = np.hstack([XS, np.ones((len(XS), 1))])
    M = 2.0 / len(XS) * Xt.T @ Xt                        # (n0+1) x (n0+1)
    n = p["n"]
    G = np.eye(n) / p["C"]
    pos = lambda j, t: j * n0 + t if t < n0 else n0 * K + j   # theta position of (w_tj | b_j)
    for j in range(K):
        for t in range(n0 + 1):
            for s in range(n0 + 1):
                G[pos(j, t), pos(j, s)] += M[t, s]
    assert np.allclose(orc.gauss_newton_dense(p["theta"], p["widths"], p["C"], XS), G, rtol=1e-13, atol=1e-15)
    v = p["v"].astype(np.float64)
    assert np.allclose(orc.Gv(p["theta"], p["widths"], p["C"], XS, v), G @ v, rtol=1e-13)


def test_no_hidden_layer_G_is_exact_hessian():
    # the second-derivative term of Eq. (hessiantogauss) vanishes for a linear model, so with
    # S = all rows G v is the derivative of grad f along v (f is quadratic: FD exact to rounding)
    p = wl.make_custom([5, 3], 30, 30, 1.3, seed=8, x="normal", n_vec=1)
    th = p["theta"].astype(np.float64)
    v = p["v"].astype(np.float64)
    g = lambda t: orc.grad(t, p["widths"], p["C"], p["X"], p["Y"])
    fd = (g(th + 0.5 * v) - g(th - 0.5 * v))
    assert np.allclose(orc.Gv(th, p["widths"], p["C"], p["X"], v), fd, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("widths", [(5, 4, 3, 2), (4, 3), (3, 5, 1), (2, 3, 3, 3, 2)])
def test_matrix_form_matches_definition(widths):
    p = tiny(widths=widths, seed=13)
    XS = p["X"][p["idx"]]
    v = p["v"].astype(np.float64)
    a = orc.Gv(p["theta"], p["widths"], p["C"], XS, v)
    b = orc.Gv_definition(p["theta"], p["widths"], p["C"], XS, v)
    G = orc.gauss_newton_dense(p["theta"], p["widths"], p["C"], XS)
    assert np.linalg.norm(a - b) <= 1e-12 * np.linalg.norm(b)
    assert np.linalg.norm(G @ v - b) <= 1e-12 * np.linalg.norm(b)
    # J v itself, row by row
    Z = orc.forward(p["theta"], p["widths"], XS)
    JV = orc.Jv(p["theta"], p["widths"], Z, v)
    for i, x in enumerate(XS):
        assert np.allclose(JV[i], orc.jacobian(p["theta"], p["widths"], x) @ v, rtol=1e-11, atol=1e-13)


def test_duplicated_rows_count_twice():
    p = tiny()
    idx = np.array([1, 1, 4], dtype=np.int32)
    v = p["v"].astype(np.float64)
    a = orc.Gv(p["theta"], p["widths"], p["C"], p["X"][idx], v)
    g1 = orc.Gv(p["theta"], p["widths"], 1e300, p["X"][[1]], v)
    g4 = orc.Gv(p["theta"], p["widths"], 1e300, p["X"][[4]], v)
    assert np.allclose(a, v / p["C"] + (2 * g1 + g4) / 3.0, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ block-diagonal (Eq. gausshat / approx-jaco)
@pytest.mark.parametrize("widths", [(5, 4, 3, 2), (3, 5, 1), (2, 3, 3, 3, 2)])
def test_blockdiag_is_G_with_offdiagonal_layer_blocks_zeroed(widths):
    p = tiny(widths=widths, seed=17)
    XS = p["X"][p["idx"]]
    v = p["v"].astype(np.float64)
    G = orc.gauss_newton_dense(p["theta"], p["widths"], p["C"], XS)
    H = orc.block_diagonal_of(G, p["widths"])
    a = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, v)
    b = orc.Gv_blockdiag_definition(p["theta"], p["widths"], p["C"], XS, v)
    assert np.linalg.norm(a - H @ v) <= 1e-12 * np.linalg.norm(H @ v)
    assert np.linalg.norm(b - H @ v) <= 1e-12 * np.linalg.norm(H @ v)
    assert np.linalg.norm(a - G @ v) > 1e-3 * np.linalg.norm(G @ v)     # it is an approximation
    assert np.allclose(H, H.T) and np.linalg.eigvalsh(H).min() >= 1.0 / p["C"] - 1e-12


def test_blockdiag_agrees_with_full_product_on_a_single_layer_direction():
    p = tiny()
    XS = p["X"][p["idx"]]
    blocks = orc.block_slices(p["widths"])
    for sl in blocks:
        v = np.zeros(p["n"])
        v[sl] = p["v"][sl]
        full = orc.Gv(p["theta"], p["widths"], p["C"], XS, v)
        hat = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, v)
        assert np.allclose(hat[sl], full[sl], rtol=1e-12, atol=1e-14)
        for other in blocks:
            if other is not sl:
                assert np.all(hat[other] == 0.0)


# ------------------------------------------------------------------ CG (Eq. full-gaussnewton, CG-stopping-cond)
def test_cg_reaches_the_dense_solution():
    p = tiny(widths=(3, 2, 2), l=10, nS=6, seed=19)
    XS = p["X"][p["idx"]]
    th = p["theta"].astype(np.float64)
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    lam = 1.0
    G = orc.gauss_newton_dense(th, p["widths"], p["C"], XS)
    n = p["n"]
    d, its, res = orc.cg_solve(th, p["widths"], p["C"], XS, g, lam, False, n, 0.0)
    exact = np.linalg.solve(G + lam * np.eye(n), -g)
    assert np.linalg.norm(d - exact) <= 1e-10 * np.linalg.norm(exact)
    # the quadratic model decreases monotonically along the iterates
    A = G + lam * np.eye(n)
    model = [0.5 * x @ A @ x + g @ x for x in its]
    assert all(b <= a + 1e-13 * abs(a) for a, b in zip([0.0] + model[:-1], model))
    assert model[0] < 0 and model[3] < model[0]
    # recorded residual norms are the true residual norms ||A d + g|| (the left side of the stop rule)
    for k, x in enumerate(its[:6], start=1):
        assert res[k][0] == pytest.approx(np.linalg.norm(A @ x + g), rel=1e-8, abs=1e-14)


def test_cg_residuals_are_mutually_orthogonal():
    p = tiny(widths=(3, 2, 2), l=10, nS=6, seed=19)
    XS = p["X"][p["idx"]]
    th = p["theta"].astype(np.float64)
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    G = orc.gauss_newton_dense(th, p["widths"], p["C"], XS) + np.eye(p["n"])
    _, its, _ = orc.cg_solve(th, p["widths"], p["C"], XS, g, 1.0, False, 3, 0.0)   # later residuals are rounding-sized
    rs = [-g] + [-(G @ x + g) for x in its]
    for a in range(len(rs)):
        for b in range(a):
            assert abs(rs[a] @ rs[b]) <= 1e-10 * np.linalg.norm(rs[a]) * np.linalg.norm(rs[b]) + 1e-20


def test_cg_stop_rule_and_first_step():
    p = tiny()
    XS = p["X"][p["idx"]]
    th = p["theta"].astype(np.float64)
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    sigma = 1e-3
    d, its, res = orc.cg_solve(th, p["widths"], p["C"], XS, g, 1.0, False, 250, sigma)
    assert len(its) < 250
    assert res[-1][0] <= sigma * np.linalg.norm(g) < res[-2][0]
    A = lambda x: orc.Gv(th, p["widths"], p["C"], XS, x) + x
    assert np.linalg.norm(A(d) + g) <= sigma * np.linalg.norm(g) * (1 + 1e-6)
    # first iterate is the exact line minimiser along -g
    alpha = (g @ g) / (g @ A(g))
    assert np.allclose(its[0], -alpha * g, rtol=1e-12)


def test_block_cg_solves_each_layer_system_on_its_own():
    p = tiny(widths=(3, 2, 2), l=10, nS=6, seed=23)
    XS = p["X"][p["idx"]]
    th = p["theta"].astype(np.float64)
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    lam = 0.5
    G = orc.gauss_newton_dense(th, p["widths"], p["C"], XS)
    d, its, res = orc.cg_solve(th, p["widths"], p["C"], XS, g, lam, True, p["n"], 0.0)
    for sl in orc.block_slices(p["widths"]):
        k = sl.stop - sl.start
        exact = np.linalg.solve(G[sl, sl] + lam * np.eye(k), -g[sl])
        assert np.linalg.norm(d[sl] - exact) <= 1e-9 * np.linalg.norm(exact)
    # per-block stop: with a tolerance, blocks stop at different steps and stay frozen
    d2, its2, res2 = orc.cg_solve(th, p["widths"], p["C"], XS, g, lam, True, 50, 1e-2)
    blocks = orc.block_slices(p["widths"])
    for b, sl in enumerate(blocks):
        gn = np.linalg.norm(g[sl])
        hit = next(k for k, r in enumerate(res2) if r[b] <= 1e-2 * gn)
        for k in range(hit, len(res2)):
            assert res2[k][b] == res2[hit][b]
        Ab = G[sl, sl] + lam * np.eye(sl.stop - sl.start)
        assert np.linalg.norm(Ab @ d2[sl] + g[sl]) <= 1e-2 * gn * (1 + 1e-9)


# ------------------------------------------------------------------ cost model (Section 4.2 / 5.2)
def test_cost_formula_fixture():
    """MACs per row of the layer GEMMs, from Eq. (jv-comp-cost) with one partition per layer."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "cost_model.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    for name, fwd, full, paper_block in rows:
        w = wl.WORKLOADS[name]["widths"]
        g = [w[m - 1] * w[m] for m in range(1, len(w))]
        assert sum(g) == int(fwd)
        assert 2 * g[0] + 4 * sum(g[1:]) == int(full)
        assert sum(2 * g[m - 1] + 2 * w[-1] * w[m] for m in range(1, len(w))) == int(paper_block)


def test_scalar_output_with_plus_minus_one_labels():
    # Section 8.3: n_L = 1, y in {-1, +1}.  f(0) = mean y^2 = 1 again, and the gradient still matches differences of f
    p = wl.make("binary300", l=40, nS=10)
    assert set(np.unique(p["Y"]).tolist()) <= {-1.0, 1.0} and p["Y"].shape == (40, 1)
    assert orc.fun(np.zeros(p["n"]), p["widths"], p["C"], p["X"], p["Y"]) == pytest.approx(1.0)
    th = p["theta"].astype(np.float64)
    g = orc.grad(th, p["widths"], p["C"], p["X"], p["Y"])
    rng = np.random.Generator(np.random.PCG64(3))
    for _ in range(5):
        e = rng.standard_normal(p["n"])
        h = 1e-6
        fd = (orc.fun(th + h * e, p["widths"], p["C"], p["X"], p["Y"]) - orc.fun(th - h * e, p["widths"], p["C"], p["X"], p["Y"])) / (2 * h)
        assert fd == pytest.approx(g @ e, rel=1e-6)


@pytest.mark.parametrize("widths", [(5, 4, 3, 2), (3, 5, 1), (2, 3, 3, 3, 2), (4, 3)])
def test_stored_factor_form_of_the_blockdiag_product(widths):
    # Section 3.3.1 / 4.2: the product through stored d z^L / d s^m equals the explicit-Jacobian definition,
    # and the factors are the Jacobian's bias columns (Eq. xtow-jaco-bias: d z^L_u / d b^m_j = d z^L_u / d s^m_j)
    p = tiny(widths=widths, seed=29)
    XS = p["X"][p["idx"]]
    v = p["v"].astype(np.float64)
    a = orc.Gv_blockdiag_stored(p["theta"], p["widths"], p["C"], XS, v)
    b = orc.Gv_blockdiag_definition(p["theta"], p["widths"], p["C"], XS, v)
    assert np.linalg.norm(a - b) <= 1e-12 * np.linalg.norm(b)
    Z = orc.forward(p["theta"], p["widths"], XS)
    D = orc.jacobian_factors(p["theta"], p["widths"], Z)
    J = orc.jacobian(p["theta"], p["widths"], XS[2])
    for m, sl in enumerate(orc.block_slices(p["widths"]), start=1):
        nm = p["widths"][m]
        assert np.allclose(D[m - 1][2], J[:, sl.stop - nm: sl.stop], rtol=1e-12, atol=1e-15)
