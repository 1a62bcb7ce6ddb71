"""CUDA path against the float64 checker, element by element, through the C ABI."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc

pytestmark = pytest.mark.gpu

# relative L2.  "fp32": FP32-accurate mode as it comes (error-compensated tensor-core contractions where the shape
# allows, FP32 FMA elsewhere); "fma": the same mode with every contraction on the FP32 FMA GEMM; "tf32": TF32 mode.
TOL = {"fp32": 1e-5, "fma": 1e-5, "tf32": 2e-3}


def rel(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return np.linalg.norm(a - b) / np.linalg.norm(b)


def relb(a, b, widths):
    """Largest relative L2 error over the whole vector and over every W^m run and every b^m run of the Section 2.1
    layout taken apart: the bias blocks and the n_L-wide output layer come from other kernels than the large weight
    blocks and are a fraction of a percent of the vector, so one norm over all n coordinates would hide them."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    worst = rel(a, b)
    for w_off, b_off, end in wl.layer_offsets(widths):
        for lo, hi in ((w_off, b_off), (b_off, end)):
            worst = max(worst, rel(a[lo:hi], b[lo:hi]))
    return worst


def make_ctx(p, mode="fp32"):
    import torch
    import paper_1802_00130_b200 as gn
    dev = torch.device("cuda:0")
    X = torch.from_numpy(p["X"]).to(dev)
    Y = torch.from_numpy(p["Y"]).to(dev)
    ctx = gn.GnContext(p["widths"], p["C"], X, Y, gn.GN_TF32 if mode == "tf32" else gn.GN_FP32_ACCURATE)
    if mode == "fma":
        ctx.set_accurate_method(1)
    ctx.set_theta(torch.from_numpy(p["theta"]).to(dev))
    return ctx


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")


SMALL = ["tiny", "ragged", "single", "mid", "binary300"]


@pytest.mark.parametrize("mode", ["fp32", "fma", "tf32"])
@pytest.mark.parametrize("name", SMALL)
def test_small_workloads_all_quantities(name, mode):
    p = wl.make(name)
    ctx = make_ctx(p, mode)
    th, w, C = p["theta"], p["widths"], p["C"]
    XS = p["X"][p["idx"]]
    ctx.set_subsample(dev(p["idx"]))
    # stored forward pass (Eq. xtoz)
    Zo = orc.forward(th, w, XS)
    for m in range(1, len(w)):
        assert rel(ctx.debug_activations(m).cpu().numpy(), Zo[m]) <= TOL[mode]
    # f and gradient over all rows
    f = ctx.fun()
    assert abs(f - orc.fun(th, w, C, p["X"], p["Y"])) <= TOL[mode] * abs(f)
    g, f2 = ctx.grad(with_f=True)
    assert abs(f2 - f) <= 1e-12 * abs(f)
    assert relb(g.cpu().numpy(), orc.grad(th, w, C, p["X"], p["Y"]), p["widths"]) <= TOL[mode]
    # products
    out = ctx.Gv(dev(p["v"])).cpu().numpy()
    assert relb(out, orc.Gv(th, w, C, XS, p["v"]), p["widths"]) <= TOL[mode]
    outb = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()
    assert relb(outb, orc.Gv_blockdiag(th, w, C, XS, p["v"]), p["widths"]) <= TOL[mode]
    ctx.close()


def test_tiny_against_explicit_jacobians():
    p = wl.make("tiny")
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    a = orc.Gv_definition(p["theta"], p["widths"], p["C"], XS, p["v"])
    b = orc.Gv_blockdiag_definition(p["theta"], p["widths"], p["C"], XS, p["v"])
    assert relb(ctx.Gv(dev(p["v"])).cpu().numpy(), a, p["widths"]) <= 1e-5
    assert relb(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy(), b, p["widths"]) <= 1e-5
    ctx.close()


@pytest.mark.parametrize("rows", [1, 7, 100, 333, 100000])
def test_row_batches_give_the_same_f_and_gradient(rows):
    p = wl.make("ragged")
    ctx = make_ctx(p)
    ctx.set_batch_rows(rows)
    g, f = ctx.grad(with_f=True)
    assert abs(f - orc.fun(p["theta"], p["widths"], p["C"], p["X"], p["Y"])) <= 1e-5 * abs(f)
    assert relb(g.cpu().numpy(), orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]), p["widths"]) <= 1e-5
    assert abs(ctx.fun() - f) <= 1e-12 * abs(f)
    ctx.close()


@pytest.mark.parametrize("blockdiag", [False, True])
@pytest.mark.parametrize("name", ["tiny", "ragged"])
def test_cg_iterates_follow_the_checker(name, blockdiag):
    p = wl.make(name)
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    d_ref, its_ref, res_ref = orc.cg_solve(p["theta"], p["widths"], p["C"], XS, g, 1.0, blockdiag, 10, 0.0)
    d, its, res, iterates = ctx.cg_solve(dev(g), 1.0, blockdiag=blockdiag, max_iter=10, tol=0.0, keep_iterates=True)
    assert its == 10 == len(its_ref)
    iterates = iterates.cpu().numpy()
    for k in range(10):
        assert rel(iterates[k], its_ref[k]) <= 1e-4, k
    assert rel(d.cpu().numpy(), d_ref) <= 1e-4
    tot = [np.sqrt(np.sum(np.square(r))) for r in res_ref]
    assert np.allclose(res[:6], tot[:6], rtol=1e-3)
    ctx.close()


@pytest.mark.parametrize("blockdiag", [False, True])
def test_cg_stop_rule(blockdiag):
    p = wl.make("mid")
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    sigma = 1e-3
    d_ref, its_ref, _ = orc.cg_solve(p["theta"], p["widths"], p["C"], XS, g, 1.0, blockdiag, 250, sigma)
    d, its, res = ctx.cg_solve(dev(g), 1.0, blockdiag=blockdiag, max_iter=250, tol=sigma)
    assert abs(its - len(its_ref)) <= 1
    assert rel(d.cpu().numpy(), d_ref) <= 2e-3       # stopped at sigma = 1e-3, possibly one step apart
    # the stop rule itself, checked with the checker's operator on the library's answer
    d64 = d.cpu().numpy().astype(np.float64)
    A = (lambda x: orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, x) + x) if blockdiag else \
        (lambda x: orc.Gv(p["theta"], p["widths"], p["C"], XS, x) + x)
    r = A(d64) + g
    segs = orc.block_slices(p["widths"]) if blockdiag else [slice(0, p["n"])]
    for s in segs:
        assert np.linalg.norm(r[s]) <= sigma * np.linalg.norm(g[s]) * 1.01
    ctx.close()


def test_degenerate_subsamples():
    import torch
    p = wl.make("ragged")
    ctx = make_ctx(p)
    v = dev(p["v"])
    # a single row
    one = np.array([5], dtype=np.int32)
    ctx.set_subsample(dev(one))
    assert relb(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], p["X"][one], p["v"]), p["widths"]) <= 1e-5
    # repeated rows count once per occurrence
    dup = np.array([1, 1, 4, 7, 7, 7], dtype=np.int32)
    ctx.set_subsample(dev(dup))
    assert relb(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], p["X"][dup], p["v"]), p["widths"]) <= 1e-5
    assert relb(ctx.Gv_blockdiag(v).cpu().numpy(),
               orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], p["X"][dup], p["v"]), p["widths"]) <= 1e-5
    # S = all rows, and a larger set after a smaller one (workspace regrowth)
    allrows = np.arange(p["l"], dtype=np.int32)
    ctx.set_subsample(dev(allrows))
    assert relb(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], p["X"], p["v"]), p["widths"]) <= 1e-5
    # the host-buffer entry points give the same bits as the device ones
    a = ctx.Gv(v).cpu().numpy()
    b = ctx.Gv_host(p["v"])
    assert np.array_equal(a, b)
    ctx.close()


def test_errors_and_state():
    import paper_1802_00130_b200 as gn
    import torch
    p = wl.make("tiny")
    dev0 = torch.device("cuda:0")
    X, Y = dev(p["X"]), dev(p["Y"])
    ctx = gn.GnContext(p["widths"], p["C"], X, Y)
    v = dev(p["v"])
    with pytest.raises(gn.GnError) as e:
        ctx.Gv(v)
    assert e.value.status == 4                      # no theta
    with pytest.raises(gn.GnError) as e:
        ctx.set_subsample(dev(p["idx"]))
    assert e.value.status == 4
    ctx.set_theta(dev(p["theta"]))
    with pytest.raises(gn.GnError) as e:
        ctx.Gv(v)
    assert e.value.status == 4                      # no subsample
    bad = p["idx"].copy()
    bad[3] = p["l"]                                 # one past the end
    with pytest.raises(gn.GnError) as e:
        ctx.set_subsample(dev(bad))
    assert e.value.status == 1
    bad[3] = -1
    with pytest.raises(gn.GnError) as e:
        ctx.set_subsample(dev(bad))
    assert e.value.status == 1
    with pytest.raises(gn.GnError):
        ctx.Gv(v)                                   # still no valid subsample
    ctx.set_subsample(dev(p["idx"]))
    out = ctx.Gv(v)
    ctx.set_theta(dev(p["theta"]))                  # stored activations are stale now
    with pytest.raises(gn.GnError) as e:
        ctx.Gv(v)
    assert e.value.status == 4
    ctx.set_subsample(dev(p["idx"]))
    assert torch.equal(ctx.Gv(v), out)              # deterministic, bit for bit
    with pytest.raises(gn.GnError) as e:
        ctx.Gv(v, out=v)
    assert e.value.status == 1
    assert ctx.kernel_launches > 0 and ctx.workspace_bytes > 0
    ctx.close()


def test_symmetry_and_positive_definiteness_on_device():
    p = wl.make("mid")
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    rng = np.random.Generator(np.random.PCG64(99))
    u = rng.standard_normal(p["n"], dtype=np.float32)
    v = p["v"]
    for fn in (ctx.Gv, ctx.Gv_blockdiag):
        Gu = fn(dev(u)).cpu().numpy().astype(np.float64)
        Gv = fn(dev(v)).cpu().numpy().astype(np.float64)
        assert abs(u @ Gv - v @ Gu) <= 1e-4 * abs(u @ Gv)
        assert v @ Gv >= v.astype(np.float64) @ v / p["C"]
    ctx.close()


def test_a_timed_out_device_wait_is_reported_and_the_context_survives():
    import paper_1802_00130_b200 as gn
    p = wl.make("mid")
    ctx = make_ctx(p, "tf32")
    ctx.set_subsample(dev(p["idx"]))
    before = ctx.Gv(dev(p["v"])).clone()
    with pytest.raises(gn.GnError) as e:
        ctx.debug_timeout_probe(1.0)                 # a barrier nothing arrives on, 1 ms limit
    assert e.value.status == 5 and "bounded wait" in str(e.value)
    # the error word was cleared and the device context is intact: same product, bit for bit
    import torch
    assert torch.equal(ctx.Gv(dev(p["v"])), before)
    g, f = ctx.grad(with_f=True)                     # a synchronising call reports no stale error
    assert np.isfinite(f)
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
@pytest.mark.parametrize("name", ["tiny", "ragged", "mid", "binary300"])
def test_blockdiag_methods_agree_with_the_checker_and_each_other(name, mode):
    import paper_1802_00130_b200 as gn
    p = wl.make(name)
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    ref = orc.Gv_blockdiag_stored(p["theta"], p["widths"], p["C"], XS, p["v"])
    outs = []
    for method in (1, 2, 0):
        ctx.set_blockdiag_method(method)
        outs.append(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy())
        assert relb(outs[-1], ref, p["widths"]) <= TOL[mode], method
    assert rel(outs[0], outs[1]) <= 2 * TOL[mode]
    # a new subsample invalidates the stored factors
    ctx.set_blockdiag_method(2)
    idx2 = np.ascontiguousarray(p["idx"][::-1][: max(1, p["nS"] // 2)])
    ctx.set_subsample(dev(idx2))
    ref2 = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], p["X"][idx2], p["v"])
    assert relb(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy(), ref2, p["widths"]) <= TOL[mode]
    # block CG goes through the same product
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    d2, _, _ = ctx.cg_solve(dev(g), 1.0, blockdiag=True, max_iter=5, tol=0.0)
    ctx.set_blockdiag_method(1)
    d1, _, _ = ctx.cg_solve(dev(g), 1.0, blockdiag=True, max_iter=5, tol=0.0)
    assert rel(d2.cpu().numpy(), d1.cpu().numpy()) <= 20 * TOL[mode]
    ctx.close()


def test_stored_factors_need_a_small_output_layer():
    import paper_1802_00130_b200 as gn
    p = wl.make("single")                      # one layer: nothing to store
    ctx = make_ctx(p)
    with pytest.raises(gn.GnError) as e:
        ctx.set_blockdiag_method(2)
    assert e.value.status == 1
    with pytest.raises(gn.GnError):
        ctx.set_blockdiag_method(3)
    with pytest.raises(gn.GnError) as e:
        ctx.set_accurate_method(3)
    assert e.value.status == 1
    ctx.close()


def test_the_default_method_builds_factors_only_when_they_pay():
    """Factors are not built for a few single products, are built at the eighth on one subsample, and at once by a
    solver that may run eight or more steps."""
    p = wl.make("mid")
    ctx = make_ctx(p, "tf32")
    ctx.set_subsample(dev(p["idx"]))
    ref = orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], p["X"][p["idx"]], p["v"])
    out = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()          # first product: the product's own scratch
    base = ctx.workspace_bytes
    for k in range(6):
        out = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()
        assert ctx.workspace_bytes == base, k
    assert relb(out, ref, p["widths"]) <= TOL["tf32"]
    out8 = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()          # eighth product: factors built and used
    grown = ctx.workspace_bytes
    factor_bytes = sum(p["nS"] * p["widths"][-1] * n for n in p["widths"][1:-1]) * 4
    assert grown - base >= factor_bytes
    assert relb(out8, ref, p["widths"]) <= TOL["tf32"]
    ctx.close()

    ctx = make_ctx(p, "tf32")
    ctx.set_subsample(dev(p["idx"]))
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    ctx.cg_solve(dev(g), 1.0, blockdiag=True, max_iter=3, tol=0.0)
    short = ctx.workspace_bytes
    ctx.cg_solve(dev(g), 1.0, blockdiag=True, max_iter=8, tol=0.0)
    assert ctx.workspace_bytes - short >= factor_bytes
    ctx.cg_solve(dev(g), 1.0, blockdiag=False, max_iter=8, tol=0.0)
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_sparse_initialisation_of_the_paper(mode):
    """Section 6.2: ceil(sqrt(n_{m-1})) N(0,1) weights into every neuron, the rest zero (saturating pre-activations)."""
    p = wl.make_custom([784, 300, 300, 10], l=2000, nS=1000, C=20.0, seed=31, x="sparse80", theta="sparse")
    w = p["widths"]
    W1 = p["theta"][: 784 * 300].reshape(300, 784)
    assert ((W1 != 0).sum(axis=1) == 28).all()                 # ceil(sqrt(784)) per neuron
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    assert relb(ctx.Gv(dev(p["v"])).cpu().numpy(), orc.Gv(p["theta"], w, p["C"], XS, p["v"]), p["widths"]) <= TOL[mode]
    assert relb(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy(), orc.Gv_blockdiag(p["theta"], w, p["C"], XS, p["v"]), p["widths"]) <= TOL[mode]
    g, f = ctx.grad(with_f=True)
    assert abs(f - orc.fun(p["theta"], w, p["C"], p["X"], p["Y"])) <= TOL[mode] * abs(f)
    assert relb(g.cpu().numpy(), orc.grad(p["theta"], w, p["C"], p["X"], p["Y"]), p["widths"]) <= TOL[mode]
    ctx.close()


def test_accurate_mode_methods_agree():
    """FP32-accurate mode on the tensor cores (hi/lo TF32 parts, chunked accumulation) against the FP32 FMA GEMM:
    both within the bound of the mode, and within twice that of each other; a new theta and a new subsample
    refresh the cached parts."""
    p = wl.make("mid")
    w, C = p["widths"], p["C"]
    outs = {}
    for mode in ("fp32", "fma"):
        ctx = make_ctx(p, mode)
        ctx.set_subsample(dev(p["idx"]))
        XS = p["X"][p["idx"]]
        a = ctx.Gv(dev(p["v"])).cpu().numpy()
        assert relb(a, orc.Gv(p["theta"], w, C, XS, p["v"]), p["widths"]) <= TOL[mode]
        # second theta, second subsample on the same context
        rng = np.random.Generator(np.random.PCG64(7))
        th2 = (p["theta"] * (1.0 + 0.1 * rng.standard_normal(p["n"]))).astype(np.float32)
        ctx.set_theta(dev(th2))
        idx2 = np.ascontiguousarray(p["idx"][::-1][: p["nS"] - 3])
        ctx.set_subsample(dev(idx2))
        b = ctx.Gv(dev(p["v"])).cpu().numpy()
        assert relb(b, orc.Gv(th2, w, C, p["X"][idx2], p["v"]), p["widths"]) <= TOL[mode]
        g = ctx.grad().cpu().numpy()
        assert relb(g, orc.grad(th2, w, C, p["X"], p["Y"]), p["widths"]) <= TOL[mode]
        outs[mode] = (a, b, g)
        ctx.close()
    for x, y in zip(outs["fp32"], outs["fma"]):
        assert rel(x, y) <= 2e-5


def test_accurate_mode_regrows_its_operand_parts_with_the_subsample():
    """A larger subsample after a smaller one moves the stored activations; the hi/lo parts cached for the old
    buffers must be dropped (no stale parts, no memory left behind)."""
    p = wl.make("mid")
    w, C = p["widths"], p["C"]
    v = dev(p["v"])
    small = np.ascontiguousarray(p["idx"][: p["nS"] // 2])
    ctx = make_ctx(p, "fp32")
    ctx.set_subsample(dev(small))
    assert relb(ctx.Gv(v).cpu().numpy(), orc.Gv(p["theta"], w, C, p["X"][small], p["v"]), p["widths"]) <= TOL["fp32"]
    ctx.set_subsample(dev(p["idx"]))
    ref = orc.Gv(p["theta"], w, C, p["X"][p["idx"]], p["v"])
    assert relb(ctx.Gv(v).cpu().numpy(), ref, p["widths"]) <= TOL["fp32"]
    grown = ctx.workspace_bytes
    ctx.close()
    fresh = make_ctx(p, "fp32")
    fresh.set_subsample(dev(p["idx"]))
    assert relb(fresh.Gv(v).cpu().numpy(), ref, p["widths"]) <= TOL["fp32"]
    assert grown <= fresh.workspace_bytes
    fresh.close()


@pytest.mark.parametrize("widths", [[20, 256, 64, 4], [784, 128, 64, 10], [100, 300, 100, 3]])
def test_accurate_mode_splits_every_operand_it_contracts(widths):
    """Networks whose weight block of a layer goes to another kernel than its activation gradient (17 <= n_m <= 128
    under a layer of >= 128 neurons): the hi / lo parts of delta s^m that the error-compensated kernel contracts must
    be those of this product, not the ones a previous product left behind.  Two products with different directions,
    then ten CG steps (every step after the first would reuse stale parts)."""
    p = wl.make_custom(widths, l=900, nS=400, C=9.0, seed=77, x="uniform", n_vec=2)
    ctx = make_ctx(p, "fp32")
    ctx.set_subsample(dev(p["idx"]))
    XS = p["X"][p["idx"]]
    th, w, C = p["theta"], p["widths"], p["C"]
    for v in (p["vs"][0], p["vs"][1], p["vs"][0]):
        assert relb(ctx.Gv(dev(v)).cpu().numpy(), orc.Gv(th, w, C, XS, v), w) <= 1e-5
    g = orc.grad(th, w, C, p["X"], p["Y"]).astype(np.float32)
    assert relb(ctx.grad().cpu().numpy(), g, w) <= 1e-5
    _, its_ref, _ = orc.cg_solve(th, w, C, XS, g, 1.0, False, 10, 0.0)
    _, its, _, iterates = ctx.cg_solve(dev(g), 1.0, blockdiag=False, max_iter=10, tol=0.0, keep_iterates=True)
    assert its == 10
    for k in range(10):
        assert rel(iterates[k].cpu().numpy(), its_ref[k]) <= 1e-4, k
    ctx.close()
