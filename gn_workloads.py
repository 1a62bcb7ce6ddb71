"""Seeded synthetic inputs for the subsampled Gauss-Newton product path.

This module only draws random numbers and shapes them; it contains none of the
method's arithmetic, so both the float64 checker and the CUDA library may be fed
from it without sharing any computation.

Every workload is a dict of numpy arrays in the layouts the C ABI expects:

    X      float32 [l][n_0]   row-major feature rows
    labels int64   [l]        class of each row
    Y      float32 [l][n_L]   one-hot label rows (Section 1 of the paper), or one column of -1 / +1
                              for the two-class, scalar-output setting (Section 8.3)
    theta  float32 [n]        model vector, per layer: columns of W^m concatenated,
                              then b^m (Section 2.1)
    idx    int32   [|S|]      subsample, drawn without replacement
    v      float32 [n]        direction for the matrix-vector product

Draw order is fixed (X, labels, theta, idx, v) from one
numpy.random.Generator(PCG64(seed)) so that a workload is reproducible from its
name alone.
"""
from __future__ import annotations

import numpy as np

# name -> recipe.  Shapes follow the networks / data sets the paper trains
# (MNIST-like 784 features, 60 000 rows, 10 classes, mostly-zero pixels in [0,1];
# an SVHN-like 3072-feature dense image set; a wider, deeper net), the data sets
# themselves being replaced by draws of the same shape and value distribution.
WORKLOADS = {
    "tiny": dict(widths=[20, 16, 16, 4], l=256, nS=64, C=1.0, x="uniform", seed=1001),
    "mnist300": dict(widths=[784, 300, 300, 10], l=60000, nS=3000, C=600.0, x="sparse80", seed=1002),
    "svhn1000": dict(widths=[3072, 1000, 1000, 10], l=50000, nS=2500, C=50000.0, x="uniform", seed=1003),
    "mnist2000_5": dict(widths=[784, 2000, 2000, 2000, 10], l=60000, nS=3000, C=60000.0, x="sparse80", seed=1004),
    "mnist2000_20": dict(widths=[784, 2000, 2000, 2000, 10], l=60000, nS=12000, C=60000.0, x="sparse80", seed=1004),
    "mnist2000_100": dict(widths=[784, 2000, 2000, 2000, 10], l=60000, nS=60000, C=60000.0, x="sparse80", seed=1004),
    "wide4096": dict(widths=[1024, 4096, 4096, 4096, 4096, 100], l=200000, nS=20000, C=200000.0, x="normal", seed=1005),
    # reduced-row relatives used where the float64 checker must finish in seconds
    "ragged": dict(widths=[37, 53, 19, 7], l=333, nS=131, C=3.0, x="sparse80", seed=1011),
    "mid": dict(widths=[200, 260, 140, 10], l=3000, nS=700, C=30.0, x="sparse80", seed=1012),
    "single": dict(widths=[50, 6], l=400, nS=150, C=2.0, x="normal", seed=1013),
    # scalar output with labels -1 / +1 (the paper's two-class setting of Section 8.3), HIGGS-like shape
    "binary300": dict(widths=[28, 300, 300, 1], l=20000, nS=2000, C=20000.0, x="normal", seed=1014, y="pm1"),
}


def num_params(widths):
    """n = sum_m (n_{m-1} n_m + n_m)."""
    return int(sum(widths[m - 1] * widths[m] + widths[m] for m in range(1, len(widths))))


def layer_offsets(widths):
    """Offsets of (w^m, b^m) inside theta: list of (w_off, b_off, end) for m = 1..L."""
    out, off = [], 0
    for m in range(1, len(widths)):
        w_off = off
        b_off = w_off + widths[m - 1] * widths[m]
        off = b_off + widths[m]
        out.append((w_off, b_off, off))
    return out


def draw_rows(rng, kind, rows, n0):
    if kind == "uniform":
        return rng.random((rows, n0), dtype=np.float32)
    if kind == "normal":
        return rng.standard_normal((rows, n0), dtype=np.float32)
    if kind == "sparse80":
        vals = rng.random((rows, n0), dtype=np.float32)
        keep = rng.random((rows, n0), dtype=np.float32) < np.float32(0.2)
        return np.where(keep, vals, np.float32(0.0)).astype(np.float32)
    raise ValueError(kind)


def draw_theta(rng, widths):
    """Every W^m and b^m entry ~ N(0, 1/n_{m-1}) (non-zero biases on purpose)."""
    parts = []
    for m in range(1, len(widths)):
        scale = np.float32(1.0 / np.sqrt(widths[m - 1]))
        parts.append(rng.standard_normal(widths[m - 1] * widths[m], dtype=np.float32) * scale)
        parts.append(rng.standard_normal(widths[m], dtype=np.float32) * scale)
    return np.concatenate(parts).astype(np.float32)


def draw_theta_sparse(rng, widths):
    """Sparse initialisation (Section 6.2 with the count of Section 8.2): of the n_{m-1} weights into a neuron
    of layer m, ceil(sqrt(n_{m-1})) randomly chosen ones are N(0, 1), the rest zero.  The paper does not say
    what the biases start as; they are zero here."""
    parts = []
    for m in range(1, len(widths)):
        a, b = widths[m - 1], widths[m]
        k = int(np.ceil(np.sqrt(a)))
        W = np.zeros((b, a), dtype=np.float32)              # row j = the weights into neuron j (theta's layout)
        for j in range(b):
            W[j, rng.choice(a, size=k, replace=False)] = rng.standard_normal(k, dtype=np.float32)
        parts.append(W.reshape(-1))
        parts.append(np.zeros(b, dtype=np.float32))
    return np.concatenate(parts)


def make(name, l=None, nS=None, with_v=True):
    """Build the named workload; `l` / `nS` override the row counts (same recipe)."""
    rec = dict(WORKLOADS[name])
    widths = list(rec["widths"])
    l = int(rec["l"] if l is None else l)
    nS = int(rec["nS"] if nS is None else nS)
    if not 0 < nS <= l:
        raise ValueError("need 0 < nS <= l")
    rng = np.random.Generator(np.random.PCG64(rec["seed"]))
    X = draw_rows(rng, rec["x"], l, widths[0])
    if rec.get("y") == "pm1":
        labels = rng.integers(0, 2, size=l)
        Y = (2.0 * labels - 1.0).astype(np.float32).reshape(l, 1)
    else:
        labels = rng.integers(0, widths[-1], size=l)
        Y = np.zeros((l, widths[-1]), dtype=np.float32)
        Y[np.arange(l), labels] = 1.0
    theta = draw_theta(rng, widths)
    idx = rng.permutation(l)[:nS].astype(np.int32)
    n = num_params(widths)
    v = rng.standard_normal(n, dtype=np.float32) if with_v else None
    C = float(rec["C"]) if l == rec["l"] else float(rec["C"]) * l / rec["l"]
    return dict(name=name, widths=widths, l=l, nS=nS, C=C, X=X, labels=labels, Y=Y,
                theta=theta, idx=idx, v=v, n=n)


def make_custom(widths, l, nS, C, seed, x="uniform", n_vec=1, theta="dense"):
    """Free-form small problem (tests): same draw order as `make`; theta "dense" or "sparse" (Section 6.2)."""
    widths = list(widths)
    rng = np.random.Generator(np.random.PCG64(seed))
    X = draw_rows(rng, x, l, widths[0])
    labels = rng.integers(0, widths[-1], size=l)
    Y = np.zeros((l, widths[-1]), dtype=np.float32)
    Y[np.arange(l), labels] = 1.0
    theta = draw_theta(rng, widths) if theta == "dense" else draw_theta_sparse(rng, widths)
    idx = rng.permutation(l)[:nS].astype(np.int32)
    n = num_params(widths)
    vs = [rng.standard_normal(n, dtype=np.float32) for _ in range(n_vec)]
    return dict(name="custom", widths=widths, l=l, nS=nS, C=float(C), X=X, labels=labels, Y=Y,
                theta=theta, idx=idx, v=vs[0], vs=vs, n=n)
