"""Newton iteration (Algorithm 3 on one GPU) against the float64 checker's."""
import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc
from test_gpu_parity import dev, make_ctx, rel

pytestmark = pytest.mark.gpu


def subsamples(p, count, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    return [rng.permutation(p["l"])[: p["nS"]].astype(np.int32) for _ in range(count)]


@pytest.mark.parametrize("blockdiag", [True, False])
@pytest.mark.parametrize("name", ["tiny", "ragged", "mid"])
def test_iterations_follow_the_checker(name, blockdiag):
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make(name)
    ctx = make_ctx(p)                                      # FP32-accurate contractions
    theta = dev(p["theta"]).clone()
    direction = torch.zeros_like(theta)
    th_ref = p["theta"].astype(np.float64)
    d_ref = np.zeros(p["n"])
    lam = lam_ref = 1.0
    # a fixed number of CG steps (sigma = 0), so that both sides take the same number whatever the rounding
    for k, idx in enumerate(subsamples(p, 3, seed=31)):
        prm = gn.NewtonParams(lam=lam, sigma=0.0, cg_max=6, blockdiag=int(blockdiag), eta=1e-4)
        rep = ctx.newton_iter(theta, dev(idx), direction, prm)
        th_ref, d_ref, lam_ref, ref = orc.newton_iteration(th_ref, p["widths"], p["C"], p["X"], p["Y"], idx, d_ref, lam_ref,
                                                           sigma=0.0, eta=1e-4, cg_max=6, blockdiag=blockdiag)
        assert rep["cg_iters"] == ref["cg_iters"] == 6
        assert rep["alpha"] == ref["alpha"] and rep["backtracks"] == ref["backtracks"]
        assert rep["f_before"] == pytest.approx(ref["f_before"], rel=2e-5)
        assert rep["f_after"] == pytest.approx(ref["f_after"], rel=2e-5)
        assert rep["beta1"] == pytest.approx(ref["beta1"], rel=2e-3, abs=1e-4)
        assert rep["beta2"] == pytest.approx(ref["beta2"], rel=2e-3, abs=2e-3)
        assert rep["rho"] == pytest.approx(ref["rho"], rel=2e-3)
        assert rep["lambda_next"] == pytest.approx(ref["lambda_next"], rel=1e-12)
        assert rel(direction.cpu().numpy(), d_ref) <= 2e-3
        assert rel(theta.cpu().numpy(), th_ref) <= 2e-4
        lam = rep["lambda_next"]
    ctx.close()


@pytest.mark.parametrize("mode", ["fp32", "tf32"])
def test_paper_settings_decrease_f_on_the_mnist_like_network(mode):
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make("mnist300", l=6000, nS=1200)
    ctx = make_ctx(p, mode)
    theta = dev(p["theta"]).clone()
    direction = torch.zeros_like(theta)
    lam, fs = 1.0, []
    for idx in subsamples(p, 4, seed=32):
        prm = gn.NewtonParams(lam=lam)                       # sigma = 0.001, CG_max = 250, (2/3, 3/2), eps = 1e-5
        th_before = theta.clone()
        rep = ctx.newton_iter(theta, dev(idx), direction, prm)
        assert rep["gTd"] < 0 and rep["cg_iters"] >= 1
        assert rep["f_after"] <= rep["f_before"] + 1e-4 * rep["alpha"] * rep["gTd"]      # Eq. (linesearch-condition)
        assert torch.allclose(theta, th_before + rep["alpha"] * direction, rtol=0, atol=1e-6)
        assert rep["lambda_next"] == pytest.approx(orc.lm_update(lam, rep["rho"], 2 / 3, 1.5))
        # f reported by the iteration is f of the returned theta
        ctx.set_theta(theta)
        assert ctx.fun() == pytest.approx(rep["f_after"], rel=1e-6)
        lam = rep["lambda_next"]
        fs.append(rep["f_after"])
    assert all(b < a for a, b in zip(fs, fs[1:])) and fs[-1] < 0.9 * fs[0]
    ctx.close()


def test_bad_parameters_are_refused():
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make("tiny")
    ctx = make_ctx(p)
    theta = dev(p["theta"]).clone()
    direction = torch.zeros_like(theta)
    for bad in (dict(eta=1.5), dict(cg_max=0), dict(lam=-1.0)):
        with pytest.raises(gn.GnError) as e:
            ctx.newton_iter(theta, dev(p["idx"]), direction, gn.NewtonParams(**bad))
        assert e.value.status == 1
    assert torch.equal(theta, dev(p["theta"]))            # nothing was touched
    ctx.close()
