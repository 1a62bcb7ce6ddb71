"""Parity at the benchmark configurations' full sizes (the launch configuration bench.py times)."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc
from test_gpu_parity import TOL, dev, make_ctx, rel

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", ["fp32", "fma", "tf32"])
def test_mnist300_products_and_gradient_on_all_rows(mode):
    p = wl.make("mnist300")
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    v = dev(p["v"])
    assert rel(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL[mode]
    ref_b = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])
    for method in (1, 2):                  # propagate form, then the stored Jacobian factors
        ctx.set_blockdiag_method(method)
        assert rel(ctx.Gv_blockdiag(v).cpu().numpy(), ref_b) <= TOL[mode], method
    g, f = ctx.grad(with_f=True)
    assert abs(f - orc.fun(p["theta"], p["widths"], p["C"], p["X"], p["Y"])) <= TOL[mode] * abs(f)
    assert rel(g.cpu().numpy(), orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"])) <= TOL[mode]
    ctx.close()


def test_svhn1000_products_and_cg():
    p = wl.make("svhn1000", l=5000)          # all 2500 subsample rows, fewer rows for f / grad
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    v = dev(p["v"])
    assert rel(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL["fp32"]
    assert rel(ctx.Gv_blockdiag(v).cpu().numpy(),
               orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL["fp32"]
    g = ctx.grad()
    g_ref = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"])
    assert rel(g.cpu().numpy(), g_ref) <= TOL["fp32"]
    # 20 CG steps on the full system: compare the first 10 iterates
    g32 = g_ref.astype(np.float32)
    _, its_ref, _ = orc.cg_solve(p["theta"], p["widths"], p["C"], XS, g32, 1.0, False, 10, 0.0)
    d, its, res, iterates = ctx.cg_solve(dev(g32), 1.0, blockdiag=False, max_iter=20, tol=0.0, keep_iterates=True)
    assert its == 20
    # FP32 products perturb the CG scalars; on this system (condition number ~1e3 at lambda = 1) the
    # iterates follow the float64 ones to ~3e-4, the tiny configuration (test_gpu_parity) to 1e-4
    for k in range(10):
        assert rel(iterates[k].cpu().numpy(), its_ref[k]) <= 1e-3
    assert res[-1] < 1e-4 * res[0]          # residual norms are not monotone in CG, but it has converged
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "fma", "tf32"])
def test_mnist2000_headline_config_at_5_percent(mode):
    p = wl.make("mnist2000_5")
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    v = dev(p["v"])
    assert rel(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL[mode]
    ref_b = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])
    for method in (1, 2):                  # propagate form, then the stored Jacobian factors
        ctx.set_blockdiag_method(method)
        assert rel(ctx.Gv_blockdiag(v).cpu().numpy(), ref_b) <= TOL[mode], method
    ctx.close()


def test_wide4096_reduced_rows_and_properties_at_full_size():
    import torch
    # element-wise parity on the first 1500 subsample rows of the same recipe ...
    p = wl.make("wide4096", l=4000, nS=1500)
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    v = dev(p["v"])
    assert rel(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL["fp32"]
    g = ctx.grad()
    assert rel(g.cpu().numpy(), orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"])) <= TOL["fp32"]
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_bench_configuration_at_20_percent(mode):
    # the workload bench.py times by default: 784-2000-2000-2000-10, |S| = 12000 (fewer rows only for the gradient)
    p = wl.make("mnist2000_20", l=12000)
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    v = dev(p["v"])
    assert rel(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL[mode]
    ref_b = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])
    for method in (1, 2):                  # propagate form, then the stored Jacobian factors
        ctx.set_blockdiag_method(method)
        assert rel(ctx.Gv_blockdiag(v).cpu().numpy(), ref_b) <= TOL[mode], method
    ctx.close()


def properties_at_any_size(p, mode, method=1):
    """Checks that need no oracle run: symmetry, the I/C lower bound, and the block-diagonal product agreeing with
    the full one on a direction supported on a single layer (then J_m v_m = J v)."""
    import torch
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    ctx.set_blockdiag_method(method)
    rng = np.random.Generator(np.random.PCG64(123))
    n = p["n"]
    u = rng.standard_normal(n, dtype=np.float32)
    v = p["v"]
    tol = 5 * TOL[mode]
    for fn in (ctx.Gv, ctx.Gv_blockdiag):
        Gu = fn(dev(u)).double()
        Gv_ = fn(dev(v)).double()
        du, dv = dev(u).double(), dev(v).double()
        a, b = float(du @ Gv_), float(dv @ Gu)
        assert abs(a - b) <= tol * max(abs(a), abs(b), float(Gv_.norm() * du.norm()) * 1e-3)
        assert float(dv @ Gv_) >= float(dv @ dv) / p["C"] * (1 - 1e-3)
        assert bool(torch.isfinite(Gv_).all())
    offs = wl.layer_offsets(p["widths"])
    for (w_off, b_off, end) in (offs[0], offs[-1], offs[len(offs) // 2]):
        vm = np.zeros(n, dtype=np.float32)
        vm[w_off:end] = v[w_off:end]
        full = ctx.Gv(dev(vm))[w_off:end].double()
        hat = ctx.Gv_blockdiag(dev(vm))[w_off:end].double()
        assert float((full - hat).norm() / full.norm()) <= tol
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_wide4096_full_size_properties(mode):
    properties_at_any_size(wl.make("wide4096", l=20000), mode)       # all 20000 subsample rows of the recipe


@pytest.mark.parametrize("method", [1, 2])
def test_mnist2000_all_rows_properties(method):
    properties_at_any_size(wl.make("mnist2000_100"), "tf32", method)  # |S| = l = 60000; method 2 keeps 14.4 GB of factors
