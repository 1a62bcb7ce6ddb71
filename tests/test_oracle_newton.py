"""Pins for the float64 checker's Newton iteration (Algorithm 3 with one partition); no GPU."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc


def test_direction_combination_minimises_the_two_variable_model():
    # Eq. (linear-comb-now): the returned (beta1, beta2) is a stationary point of
    # q(beta) = 1/2 (b1 d + b2 dbar)^T G (b1 d + b2 dbar) + g^T (b1 d + b2 dbar), checked by finite differences of q
    rng = np.random.Generator(np.random.PCG64(5))
    n = 9
    M = rng.standard_normal((n, n))
    G = M @ M.T + np.eye(n)
    d, dbar, g = rng.standard_normal(n), rng.standard_normal(n), rng.standard_normal(n)
    b1, b2 = orc.combine_directions(d @ G @ d, dbar @ G @ d, dbar @ G @ dbar, -(g @ d), -(g @ dbar), 1e-5)
    q = lambda x, y: 0.5 * (x * d + y * dbar) @ G @ (x * d + y * dbar) + g @ (x * d + y * dbar)
    h = 1e-5
    assert abs(q(b1 + h, b2) - q(b1 - h, b2)) / (2 * h) < 1e-6
    assert abs(q(b1, b2 + h) - q(b1, b2 - h)) / (2 * h) < 1e-6
    for _ in range(20):                                   # and it is the minimum (G positive definite)
        e = rng.standard_normal(2) * 0.3
        assert q(b1 + e[0], b2 + e[1]) >= q(b1, b2)
    # Eq. (determinant): degenerate systems fall back to (1, 0); dbar = 0 is the first iteration
    assert orc.combine_directions(2.0, 0.0, 0.0, 1.0, 0.0, 1e-5) == (1.0, 0.0)
    assert orc.combine_directions(1.0, 1.0, 1.0 + 1e-7, 1.0, 1.0, 1e-5) == (1.0, 0.0)


def test_levenberg_marquardt_rule_table():
    assert orc.lm_update(3.0, 0.9, 2 / 3, 1.5) == pytest.approx(2.0)
    assert orc.lm_update(3.0, 0.75, 2 / 3, 1.5) == 3.0
    assert orc.lm_update(3.0, 0.25, 2 / 3, 1.5) == 3.0
    assert orc.lm_update(3.0, 0.2499, 2 / 3, 1.5) == pytest.approx(4.5)
    assert orc.lm_update(3.0, -5.0, 2 / 3, 1.5) == pytest.approx(4.5)


def test_linear_model_is_solved_in_one_undamped_step():
    # no hidden layer: f is quadratic and G (S = all rows) is its Hessian, so with lambda = 0 and CG run to
    # convergence the step alpha = 1 lands on the minimiser: gradient zero, rho = 1, lambda dropped
    p = wl.make_custom([5, 3], 40, 40, 1.7, seed=21, x="normal")
    th = p["theta"].astype(np.float64)
    idx = np.arange(p["l"])
    th1, d, lam1, rep = orc.newton_iteration(th, p["widths"], p["C"], p["X"], p["Y"], idx, np.zeros(p["n"]), 0.0,
                                             sigma=1e-13, cg_max=200, blockdiag=False)
    assert rep["alpha"] == 1.0 and rep["backtracks"] == 0 and (rep["beta1"], rep["beta2"]) == (1.0, 0.0)
    assert np.linalg.norm(orc.grad(th1, p["widths"], p["C"], p["X"], p["Y"])) < 1e-9
    assert rep["rho"] == pytest.approx(1.0, rel=1e-9)
    assert lam1 == 0.0


def test_iterations_decrease_f_and_respect_the_line_search():
    p = wl.make("tiny")
    th = p["theta"].astype(np.float64)
    dprev = np.zeros(p["n"])
    lam, eta = 1.0, 1e-4
    rng = np.random.Generator(np.random.PCG64(77))
    fs = [orc.fun(th, p["widths"], p["C"], p["X"], p["Y"])]
    for k in range(4):
        idx = rng.permutation(p["l"])[:64]
        th_new, d, lam_new, rep = orc.newton_iteration(th, p["widths"], p["C"], p["X"], p["Y"], idx, dprev, lam, eta=eta)
        assert rep["f_before"] == pytest.approx(fs[-1], rel=1e-14)
        # Eq. (linesearch-condition) holds at alpha and (when alpha < 1) fails at 2 alpha
        assert rep["f_after"] <= rep["f_before"] + eta * rep["alpha"] * rep["gTd"]
        assert rep["gTd"] < 0
        if rep["alpha"] < 1.0:
            f2 = orc.fun(th + 2 * rep["alpha"] * d, p["widths"], p["C"], p["X"], p["Y"])
            assert f2 > rep["f_before"] + eta * 2 * rep["alpha"] * rep["gTd"]
        assert np.allclose(th_new, th + rep["alpha"] * d)
        assert lam_new == orc.lm_update(lam, rep["rho"], 2 / 3, 1.5)
        if k == 0:
            assert (rep["beta1"], rep["beta2"]) == (1.0, 0.0)
        th, dprev, lam = th_new, d, lam_new
        fs.append(rep["f_after"])
    assert all(b < a for a, b in zip(fs, fs[1:]))
    assert fs[-1] < 0.8 * fs[0]
