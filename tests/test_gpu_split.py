"""Variable partition (Section 3.1): partition-wise block-diagonal product and its CG against the checker."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc
from test_gpu_parity import TOL, dev, make_ctx, rel

pytestmark = pytest.mark.gpu

# (workload, split): boundaries that are and are not multiples of 4, splits of the input and output layers
CASES = [("tiny", [2, 2, 2, 1]), ("tiny", [1, 3, 2, 2]), ("tiny", [4, 1, 4, 4]),
         ("ragged", None), ("mid", [2, 2, 2, 1]), ("mid", [1, 1, 5, 2]), ("mid", [3, 4, 1, 1]),
         ("binary300", [1, 2, 3, 1]), ("single", None)]


def split_for(p, split):
    if split is not None:
        return split
    w = p["widths"]                       # two groups wherever a layer has at least two neurons
    return [2 if n >= 2 else 1 for n in w]


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
@pytest.mark.parametrize("name,split", CASES)
def test_partition_product(name, split, mode):
    p = wl.make(name)
    split = split_for(p, split)
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    ctx.set_split(split)
    _, P = orc.partition_labels(p["widths"], split)
    assert ctx.num_partitions == P
    XS = p["X"][p["idx"]]
    ref = orc.Gv_partition(p["theta"], p["widths"], p["C"], XS, p["v"], split)
    out = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()
    assert rel(out, ref) <= TOL[mode]
    # per partition as well: a small partition must not hide behind a large one
    for idx in orc.partition_indices(p["widths"], split):
        assert rel(out[idx], ref[idx]) <= 2 * TOL[mode]
    # the full product is untouched by the split, and unit counts restore the layer blocks
    assert rel(ctx.Gv(dev(p["v"])).cpu().numpy(), orc.Gv(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL[mode]
    ctx.set_split([1] * len(split))
    assert ctx.num_partitions == len(split) - 1
    assert rel(ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy(),
               orc.Gv_blockdiag(p["theta"], p["widths"], p["C"], XS, p["v"])) <= TOL[mode]
    ctx.close()


@pytest.mark.parametrize("name,split", [("tiny", [2, 2, 2, 1]), ("tiny", [1, 3, 2, 2]), ("ragged", None)])
def test_partition_cg_iterates(name, split):
    p = wl.make(name)
    split = split_for(p, split)
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    ctx.set_split(split)
    XS = p["X"][p["idx"]]
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    _, its_ref, res_ref = orc.cg_partitioned(p["theta"], p["widths"], p["C"], XS, g, 1.0, split, 10, 0.0)
    d, its, res, iterates = ctx.cg_solve(dev(g), 1.0, blockdiag=True, max_iter=10, tol=0.0, keep_iterates=True)
    assert its == 10
    for k in range(10):
        assert rel(iterates[k].cpu().numpy(), its_ref[k]) <= 1e-4
    tot = np.sqrt((np.array(res_ref) ** 2).sum(axis=1))
    assert np.allclose(res, tot, rtol=1e-3)
    ctx.close()


def test_termination_rule_matches_the_checker_step_for_step():
    p = wl.make("mid")
    split = [2, 3, 2, 1]
    ctx = make_ctx(p)
    ctx.set_subsample(dev(p["idx"]))
    ctx.set_split(split)
    XS = p["X"][p["idx"]]
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    tol, lam = 1e-2, 1e-3
    counts = {}
    for cg_min, share in ((0, 1.0), (0, 0.5), (0, 0.25), (9, 0.25), (3, 0.75)):
        _, its_ref, res_ref = orc.cg_partitioned(p["theta"], p["widths"], p["C"], XS, g, lam, split, 60, tol,
                                                 cg_min=cg_min, finished_share=share)
        ctx.set_cg_termination(cg_min, share)
        d, its, res = ctx.cg_solve(dev(g), lam, blockdiag=True, max_iter=60, tol=tol)
        assert its == len(its_ref), (cg_min, share)
        assert rel(d.cpu().numpy(), its_ref[-1]) <= 2e-3
        counts[(cg_min, share)] = its
    assert counts[(0, 0.25)] < counts[(0, 1.0)]               # the rule did cut the solve short
    assert counts[(9, 0.25)] == min(9, counts[(0, 1.0)]) > counts[(0, 0.25)]    # cg_min holds the early stop back
    # the full system ignores the rule
    ctx.set_cg_termination(0, 0.25)
    _, its_full, _ = ctx.cg_solve(dev(g), lam, blockdiag=False, max_iter=5, tol=0.0)
    assert its_full == 5
    ctx.close()


def test_newton_iteration_with_a_split_structure():
    import paper_1802_00130_b200 as gn
    import torch
    p = wl.make("mid")
    split = [1, 2, 2, 1]
    ctx = make_ctx(p)
    ctx.set_split(split)
    theta = dev(p["theta"]).clone()
    dbar = torch.zeros_like(theta)
    prm = gn.NewtonParams(lam=1.0, sigma=1e-3, cg_max=30, blockdiag=1)
    rep = ctx.newton_iter(theta, dev(p["idx"]), dbar, prm)
    assert rep["f_after"] < rep["f_before"]
    assert abs(rep["f_before"] - orc.fun(p["theta"], p["widths"], p["C"], p["X"], p["Y"])) <= 1e-5 * rep["f_before"]
    assert abs(rep["f_after"] - orc.fun(theta.cpu().numpy(), p["widths"], p["C"], p["X"], p["Y"])) <= 1e-5 * rep["f_after"]
    ctx.close()


def test_bad_split_structures_are_refused():
    import paper_1802_00130_b200 as gn
    p = wl.make("tiny")
    ctx = make_ctx(p)
    for bad in ([0, 1, 1, 1], [1, 17, 1, 1], [1, 1, 1, 5]):
        with pytest.raises(gn.GnError) as e:
            ctx.set_split(bad)
        assert e.value.status == 1
    with pytest.raises(ValueError):
        ctx.set_split([1, 1])
    with pytest.raises(gn.GnError):
        ctx.set_cg_termination(0, 0.0)
    with pytest.raises(gn.GnError):
        ctx.set_cg_termination(-1, 1.0)
    assert ctx.num_partitions == 3
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_paper_style_network_784_800_800_10_split_1_1_3_1(mode):
    # the shape and split structure of the paper's 7-partition MNIST setting, on synthetic rows
    p = wl.make_custom([784, 800, 800, 10], l=3000, nS=1500, C=3000.0, seed=77, x="sparse80")
    split = [1, 1, 3, 1]
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    ctx.set_split(split)
    assert ctx.num_partitions == 7
    XS = p["X"][p["idx"]]
    ref = orc.Gv_partition(p["theta"], p["widths"], p["C"], XS, p["v"], split)
    out = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()
    assert rel(out, ref) <= TOL[mode]
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_headline_network_with_a_split_at_5_percent(mode):
    p = wl.make("mnist2000_5")
    split = [1, 2, 2, 2, 1]                                   # 1000-neuron groups: 16-byte paths throughout
    ctx = make_ctx(p, mode)
    ctx.set_subsample(dev(p["idx"]))
    ctx.set_split(split)
    assert ctx.num_partitions == 2 + 4 + 4 + 2
    XS = p["X"][p["idx"]]
    ref = orc.Gv_partition(p["theta"], p["widths"], p["C"], XS, p["v"], split)
    out = ctx.Gv_blockdiag(dev(p["v"])).cpu().numpy()
    assert rel(out, ref) <= TOL[mode]
    ctx.close()
