"""Work issued together: the independent large contractions of a layer as one launch of the CTA-pair kernel (TF32
mode), its bias column sums and n_L-row weight block on a side stream, and the consecutive layers of a pass as one
launch whose tiles wait for the tiles they read.  Same bits as one launch after the other on one stream, and the
usual bound against the float64 checker."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc
from test_gpu_parity import TOL, dev, make_ctx, relb

pytestmark = pytest.mark.gpu

CASES = {
    "mid": lambda: wl.make("mid"),
    "ragged_wide": lambda: wl.make_custom([300, 520, 392, 10], l=1500, nS=1100, C=15.0, seed=41, x="sparse80"),
    "mnist2000_5": lambda: wl.make("mnist2000_5", l=6000),
    "svhn1000": lambda: wl.make("svhn1000", l=5000),
    "deep": lambda: wl.make_custom([256, 384, 256, 512, 256, 8], l=2000, nS=1300, C=20.0, seed=43, x="uniform"),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_grouped_launches_give_the_bits_of_single_launches(name):
    import torch
    p = CASES[name]()
    outs = []
    for grouped, side, chain, back in ((0, 0, 0, 0), (1, 1, 2, 1), (1, 0, 0, 0), (0, 1, 1, 1), (0, 0, 2, 0), (0, 0, 1, 1)):
        ctx = make_ctx(p, "tf32")
        ctx.debug_option(1, 0)                  # whole tiles only in every run: K slices change the order of sums
        ctx.debug_option(0, grouped)
        ctx.debug_option(3, side)
        ctx.debug_option(4, chain)
        ctx.debug_option(8, back)               # hidden layers of a backward pass as one chained launch
        ctx.set_subsample(dev(p["idx"]))
        v = dev(p["v"])
        res = [ctx.Gv(v).clone()]
        for method in (1, 2):
            ctx.set_blockdiag_method(method)
            res.append(ctx.Gv_blockdiag(v).clone())
        res.append(ctx.grad().clone())
        for m in range(1, len(p["widths"])):        # the stored forward pass itself
            res.append(ctx.debug_activations(m).clone())
        launches = ctx.kernel_launches
        outs.append((res, launches))
        ctx.close()
    for other in outs[1:]:
        for a, b in zip(outs[0][0], other[0]):
            assert torch.equal(a, b)
    assert outs[1][1] < outs[0][1]              # fewer launches: something was in fact grouped
    XS = p["X"][p["idx"]]
    th, w, C = p["theta"], p["widths"], p["C"]
    res = [r.cpu().numpy() for r in outs[1][0]]
    assert relb(res[0], orc.Gv(th, w, C, XS, p["v"]), w) <= TOL["tf32"]
    ref_b = orc.Gv_blockdiag(th, w, C, XS, p["v"])
    assert relb(res[1], ref_b, w) <= TOL["tf32"]
    assert relb(res[2], ref_b, w) <= TOL["tf32"]
    assert relb(res[3], orc.grad(th, w, C, p["X"], p["Y"]), w) <= TOL["tf32"]


@pytest.mark.parametrize("name", ["mid", "deep", "mnist2000_5"])
def test_parts_written_by_the_epilogue_are_the_parts_a_separate_pass_would_write(name):
    """FP32-accurate mode: the error-compensated kernel writes the hi / lo TF32 parts of a result that a later
    contraction of the same product (or row batch) takes as an operand.  Same bits as splitting that result in a pass
    of its own, fewer launches, and the mode's bound against the float64 checker."""
    import torch
    p = CASES[name]()
    outs = []
    for emit in (0, 1):
        ctx = make_ctx(p, "fp32")
        ctx.debug_option(5, emit)
        ctx.set_subsample(dev(p["idx"]))
        v = dev(p["v"])
        res = [ctx.Gv(v).clone(), ctx.grad().clone(), ctx.Gv(v).clone()]
        for method in (1, 2):
            ctx.set_blockdiag_method(method)
            res.append(ctx.Gv_blockdiag(v).clone())
        res.append(ctx.Gv(v).clone())           # after the block-diagonal products have rewritten the same buffers
        outs.append((res, ctx.kernel_launches))
        ctx.close()
    for a, b in zip(outs[0][0], outs[1][0]):
        assert torch.equal(a, b)
    assert outs[1][1] < outs[0][1]
    XS = p["X"][p["idx"]]
    th, w, C = p["theta"], p["widths"], p["C"]
    res = [r.cpu().numpy() for r in outs[1][0]]
    ref = orc.Gv(th, w, C, XS, p["v"])
    for k in (0, 2, 5):
        assert relb(res[k], ref, w) <= TOL["fp32"]
    assert relb(res[1], orc.grad(th, w, C, p["X"], p["Y"]), w) <= TOL["fp32"]
    ref_b = orc.Gv_blockdiag(th, w, C, XS, p["v"])
    assert relb(res[3], ref_b, w) <= TOL["fp32"] and relb(res[4], ref_b, w) <= TOL["fp32"]


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
@pytest.mark.parametrize("name", ["tiny", "ragged", "mid"])
def test_replayed_cg_step_gives_the_bits_of_plain_launches(name, mode):
    """Fixed-length CG solves of small problems capture their second step as a CUDA graph and replay it; the graph is
    kept across solves.  Same iterates and residual norms, bit for bit, as plain launches: over two subsamples, two
    damping values and both kinds of system, with an early-stopping solve (which never uses the graph) in between."""
    import torch
    p = wl.make(name)
    g = dev(orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32))
    idx2 = np.ascontiguousarray(p["idx"][::-1])
    runs = []
    for graph in (0, 1):
        ctx = make_ctx(p, mode)
        ctx.debug_option(6, graph)
        got = []
        for idx, lam in ((p["idx"], 1.0), (idx2, 1.0), (idx2, 0.5)):
            ctx.set_subsample(dev(idx))
            for blockdiag in (False, True):
                d, its, res = ctx.cg_solve(g, lam, blockdiag=blockdiag, max_iter=9, tol=0.0)
                assert its == 9
                got.append((d.clone(), res.copy()))
            d, its, res = ctx.cg_solve(g, lam, blockdiag=True, max_iter=50, tol=1e-2)
            got.append((d.clone(), res.copy()))
        runs.append(got)
        # 6 fixed-length solves of 9 steps: the first step of each is plain, the other 8 are replays
        assert ctx.graph_replays == (6 * 8 if graph else 0)
        ctx.close()
    for (d0, r0), (d1, r1) in zip(*runs):
        assert torch.equal(d0, d1)
        assert np.array_equal(r0, r1)
    # and against the checker (first solve, full system)
    XS = p["X"][p["idx"]]
    d_ref, _, _ = orc.cg_solve(p["theta"], p["widths"], p["C"], XS, g.cpu().numpy(), 1.0, False, 9, 0.0)
    tol = 1e-4 if mode == "fp32" else 2e-2
    assert np.linalg.norm(runs[1][0][0].cpu().numpy() - d_ref) <= tol * np.linalg.norm(d_ref)


def test_a_context_on_the_callers_own_stream_gives_the_same_bits():
    """Everything is enqueued on the stream given to gn_create (here a non-default stream of the caller's; the other
    tests leave it to the context to make one): products, gradient and a graph-replayed CG solve, bit for bit."""
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make("mid")
    X, Y, th, idx, v = dev(p["X"]), dev(p["Y"]), dev(p["theta"]), dev(p["idx"]), dev(p["v"])
    g = dev(orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32))
    torch.cuda.synchronize()
    outs = []
    for own in (False, True):
        stream = torch.cuda.Stream() if own else None
        ctx = gn.GnContext(p["widths"], p["C"], X, Y, gn.GN_TF32, stream=stream)
        ctx.set_theta(th)
        ctx.set_subsample(idx)
        res = [ctx.Gv(v), ctx.Gv_blockdiag(v), ctx.grad()]
        d, its, resn = ctx.cg_solve(g, 1.0, blockdiag=False, max_iter=8, tol=0.0)
        assert its == 8 and ctx.graph_replays == 7
        res.append(d)
        torch.cuda.synchronize()
        outs.append([r.clone() for r in res] + [torch.from_numpy(resn)])
        ctx.close()
    for a, b in zip(*outs):
        assert torch.equal(a.cpu(), b.cpu())


def test_weight_blocks_of_the_stored_factor_product_in_two_chained_halves():
    """From 4096 subsample rows on, TF32 mode cuts every hidden-layer weight block of the stored-factor product into
    the two halves of the rows; the second half adds onto the first inside one chained launch.  Same result as the
    uncut blocks up to the order of two partial sums, deterministic, and within the mode's bound of the checker."""
    import torch
    p = wl.make_custom([300, 520, 392, 264, 10], l=5200, nS=5000, C=52.0, seed=47, x="sparse80")
    XS = p["X"][p["idx"]]
    ref = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])
    outs = {}
    for cut in (1, 0):
        ctx = make_ctx(p, "tf32")
        ctx.debug_option(7, cut)
        ctx.set_blockdiag_method(2)
        ctx.set_subsample(dev(p["idx"]))
        a = ctx.Gv_blockdiag(dev(p["v"])).clone()
        b = ctx.Gv_blockdiag(dev(p["v"])).clone()
        assert torch.equal(a, b)                              # deterministic
        outs[cut] = (a.cpu().numpy(), ctx.kernel_launches)
        assert relb(outs[cut][0], ref, p["widths"]) <= TOL["tf32"]
        ctx.close()
    assert not np.array_equal(outs[1][0], outs[0][0])          # the cut form did run (another order of sums)
    # ... and differs by rounding only: the tensor core adds into its FP32 accumulator with truncation (a relative bias
    # of about 1e-9 per term), so one accumulation over 5000 rows and two over 2500 differ by about 1e-5
    assert relb(outs[1][0], outs[0][0], p["widths"]) <= 1e-4


@pytest.mark.parametrize("mode", ["tf32", "fp32"])
@pytest.mark.parametrize("name", ["mid", "mnist2000_5", "svhn1000"])
def test_last_factor_formed_on_the_fly_gives_the_bits_of_the_stored_one(name, mode):
    """Stored-factor block product (Section 3.3.1 / 4.2): the factor of the last hidden layer has the closed form
    W^L * sigma'(z^{L-1}); forming it inside the per-sample kernel gives the bits of reading the stored copy back."""
    import torch
    p = CASES[name]()
    outs = []
    for fly in (0, 1):
        ctx = make_ctx(p, mode)
        ctx.debug_option(9, fly)
        ctx.set_blockdiag_method(2)
        ctx.set_subsample(dev(p["idx"]))
        outs.append(ctx.Gv_blockdiag(dev(p["v"])).clone())
        ctx.close()
    assert torch.equal(outs[0], outs[1])
    ref = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], p["X"][p["idx"]], p["v"])
    assert relb(outs[1].cpu().numpy(), ref, p["widths"]) <= TOL[mode]
