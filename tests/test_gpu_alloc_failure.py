"""Device allocations refused on the host (a test hook counts down to the allocation to refuse): every entry point
that grows a workspace must hand back GN_ENOMEM (or fall back where the method allows), keep the context usable, and
leave the memory accounting exact.  Nothing on the device faults in any of this."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc
from test_gpu_parity import dev, relb

pytestmark = pytest.mark.gpu

GN_ENOMEM = 2


def fresh(p, mode):
    import torch
    import paper_1802_00130_b200 as gn
    X, Y = dev(p["X"]), dev(p["Y"])
    ctx = gn.GnContext(p["widths"], p["C"], X, Y, gn.GN_TF32 if mode == "tf32" else gn.GN_FP32_ACCURATE)
    ctx.set_theta(dev(p["theta"]))
    return ctx


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_refused_allocations_surface_as_enomem_and_the_context_recovers(mode):
    import paper_1802_00130_b200 as gn
    p = wl.make("mid")
    w, C = p["widths"], p["C"]
    XS = p["X"][p["idx"]]
    tol = 1e-5 if mode == "fp32" else 2e-3
    ref_gv = orc.Gv(p["theta"], w, C, XS, p["v"])
    ref_gb = orc.Gv_blockdiag(p["theta"], w, C, XS, p["v"])
    ref_g = orc.grad(p["theta"], w, C, p["X"], p["Y"])

    # what a run without refusals ends up holding
    clean = fresh(p, mode)
    clean.set_subsample(dev(p["idx"]))
    clean.Gv(dev(p["v"]))
    clean.set_blockdiag_method(2)
    clean.Gv_blockdiag(dev(p["v"]))
    clean.grad()
    prm = gn.NewtonParams(lam=1.0, sigma=1e-3, cg_max=4, blockdiag=1)
    th = dev(p["theta"]).clone(); dbar = dev(np.zeros(p["n"], np.float32))
    clean.newton_iter(th, dev(p["idx"]), dbar, prm)
    clean_bytes = clean.workspace_bytes
    clean.close()

    ctx = fresh(p, mode)
    v = dev(p["v"])
    seen = 0
    ops = [
        ("set_subsample", lambda: ctx.set_subsample(dev(p["idx"]))),
        ("Gv", lambda: ctx.Gv(v)),
        ("Gv_blockdiag (stored factors)", lambda: ctx.Gv_blockdiag(v)),
        ("grad", lambda: ctx.grad()),
    ]
    ctx.set_blockdiag_method(2)
    for name, op in ops:
        n = 1
        while True:
            ctx.debug_option(2, n)
            try:
                op()
            except gn.GnError as e:
                assert e.status == GN_ENOMEM, (name, n, str(e))
                assert "refused" in str(e) or "cudaMalloc" in str(e)
                seen += 1
                n += 1
                assert n < 80
                continue
            finally:
                ctx.debug_option(2, 0)
            break                                 # ran through: either no allocation was left to refuse, or the
                                                  # method fell back (FP32-accurate mode without room for hi / lo parts)
        op()                                      # and now without the hook
    assert seen >= 8                              # the walk did meet allocations in every stage
    assert relb(ctx.Gv(v).cpu().numpy(), ref_gv, w) <= tol
    assert relb(ctx.Gv_blockdiag(v).cpu().numpy(), ref_gb, w) <= tol
    assert relb(ctx.grad().cpu().numpy(), ref_g, w) <= tol

    # the Newton iteration: refuse its n-th allocation, then run it clean and compare with a fresh context
    th = dev(p["theta"]).clone(); dbar = dev(np.zeros(p["n"], np.float32))
    n = 1
    while True:
        ctx.debug_option(2, n)
        th.copy_(dev(p["theta"])); dbar.zero_()
        try:
            rep = ctx.newton_iter(th, dev(p["idx"]), dbar, prm)
        except gn.GnError as e:
            assert e.status == GN_ENOMEM
            n += 1
            assert n < 40
            continue
        finally:
            ctx.debug_option(2, 0)
        break
    other = fresh(p, mode)
    other.set_blockdiag_method(2)
    th2 = dev(p["theta"]).clone(); dbar2 = dev(np.zeros(p["n"], np.float32))
    rep2 = other.newton_iter(th2, dev(p["idx"]), dbar2, prm)
    assert abs(rep["f_after"] - rep2["f_after"]) <= 1e-6 * abs(rep2["f_after"])
    assert rep["cg_iters"] == rep2["cg_iters"]
    other.close()
    # accounting: what this context holds is what its allocations add up to; no more than a clean run plus the
    # fall-back buffers it may have kept, and all of it goes away with the context
    assert ctx.workspace_bytes <= 1.5 * clean_bytes
    ctx.close()
    again = fresh(p, mode)
    again.set_subsample(dev(p["idx"]))
    again.Gv(v)
    again.set_blockdiag_method(2)
    again.Gv_blockdiag(v)
    again.grad()
    th = dev(p["theta"]).clone(); dbar = dev(np.zeros(p["n"], np.float32))
    again.newton_iter(th, dev(p["idx"]), dbar, prm)
    assert again.workspace_bytes == clean_bytes   # a context created after all that grows to exactly the clean size
    again.close()


def test_a_refused_split_structure_leaves_the_old_one_in_force():
    import paper_1802_00130_b200 as gn
    p = wl.make("mid")
    ctx = fresh(p, "fp32")
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    ref = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    refused = 0
    for n in range(1, 10):
        ctx.debug_option(2, n)
        try:
            ctx.set_split([1, 2, 2, 1])
        except gn.GnError as e:
            assert e.status == GN_ENOMEM
            refused += 1
            ctx.debug_option(2, 0)
            assert ctx.num_partitions == 3                   # still one block per layer, and its tables still work
            d, its, res = ctx.cg_solve(dev(g), 1.0, blockdiag=True, max_iter=3, tol=0.0)
            assert its == 3
            assert relb(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy(), ref, p["widths"]) <= 1e-5
            continue
        finally:
            ctx.debug_option(2, 0)
        break
    assert refused >= 2
    assert ctx.num_partitions == 1 * 2 + 2 * 2 + 2 * 1       # the call that was let through took effect
    ctx.set_split([1, 1, 1, 1])
    assert relb(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy(), ref, p["widths"]) <= 1e-5
    ctx.close()
