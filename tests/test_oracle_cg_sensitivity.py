"""How far CG iterates move when every product carries a relative error of the size an FP32 contraction has.

No GPU code runs here.  The checker's own CG (Eq. sample-gaussnewton, textbook recurrences) is run twice on the
3072-1000-1000-10 system at lambda = 1: once in float64, once with every product it receives perturbed by a seeded
relative error and rounded to float32.  The third Lanczos step of this system is ill conditioned: the perturbation
is amplified a few hundred times there and the deviation then stays.  This fixes, from the checker alone, the bound
the device test may use for the CG iterates of this configuration: amplification x the product error it asserts.
"""
import numpy as np

import gn_workloads as wl
from oracle import gn_oracle as orc


def rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


# ceiling of the amplification this test measures; tests/test_gpu_fullsize.py multiplies it by the product error
# it has just asserted on the device to bound the device's CG iterates on the same system
AMPLIFICATION_BOUND = 600.0


def perturbed_cg(p, XS, g, eps, steps, seed=5):
    rng = np.random.Generator(np.random.PCG64(seed))
    th, w, C = p["theta"], p["widths"], p["C"]

    def product(x):
        q = orc.Gv(th, w, C, XS, x.astype(np.float32).astype(np.float64))   # the direction as float32 holds it
        q = q * (1.0 + eps * rng.standard_normal(q.size))                      # relative L2 error eps
        return q.astype(np.float32).astype(np.float64)                         # the product as float32 holds it

    return orc.cg(product, g, 1.0, steps, 0.0)


def test_fp32_sized_product_errors_move_the_svhn1000_iterates_by_hundreds_of_times_their_size():
    p = wl.make("svhn1000", l=5000)
    XS = p["X"][p["idx"]]
    g = orc.grad(p["theta"], p["widths"], p["C"], p["X"], p["Y"]).astype(np.float32)
    steps = 6
    _, exact, res = orc.cg(lambda x: orc.Gv(p["theta"], p["widths"], p["C"], XS, x), g, 1.0, steps, 0.0)
    eps = 7e-7                                            # relative L2 error of one FP32-accurate product
    _, moved, _ = perturbed_cg(p, XS, g, eps, steps)
    dev = [rel(moved[k], exact[k]) for k in range(steps)]
    # the first two iterates see the error at its own size, the third amplifies it, later ones keep it
    assert dev[0] <= 2 * eps and dev[1] <= 4 * eps
    assert dev[2] >= 1e-4                                 # so 1e-4 cannot hold here for any product of that accuracy
    assert max(dev) / eps <= AMPLIFICATION_BOUND
    assert max(dev) / eps >= 100.0
    assert abs(dev[5] - dev[3]) <= 0.2 * dev[3]           # no further growth
    # the residual norms are not monotone on this system (step 3 goes up): the history is what CG does, not an error
    tot = [float(r[0]) for r in res]
    assert tot[3] > tot[2]
