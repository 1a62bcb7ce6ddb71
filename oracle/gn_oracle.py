"""Float64 CPU checker for the subsampled Gauss-Newton product path.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow statement of what the
CUDA library must compute, written from the paper ("Distributed Newton Methods
for Deep Neural Networks", arXiv 1802.00130).  It shares no code with the CUDA
path and must never be imported by it; only tests, the smoke check and the
benchmark's CPU-baseline leg call it.

Two tiers:

* tier D ("definition"): explicit per-sample Jacobians J^i built with the
  paper's backward recurrence (Section 3.3), the dense Gauss-Newton matrix
  (Eq. def-gauss-newton / sampled-Gauss), its block-diagonal version
  (Eq. gausshat) - tiny inputs only.
* tier M ("matrix form"): the same quantities for all rows at once in float64
  matrix form (forward directional derivative for J v, the back-propagation
  equations of Section 2.2 for J^T u).  Usable at the paper's network sizes.

Pins (see tests/test_oracle_pins.py): f(0) closed form, a hand-computed 2-1-1
network, finite differences of f and of the network output, symmetry and
positive-definiteness of G, the closed form of G for a network with no hidden
layer, the exact-Hessian property in that case, tier M against tier D, dense
solves for CG.  The paper prints no numeric worked example of f, grad f, J or
G v, so beyond those pins the values are unpinned by the paper itself.

Readings of the paper taken here (each is also listed in the design notes):
biases are part of theta and are regularised (Section 3.2.1 sums (b_j)^2 into
the regulariser); the loss has no 1/2 so B^i = 2I (Section 3.1); f and grad f
average over all l rows, G^S over |S|; the Jacobian's backward pass starts from
the identity (Eq. zLindependent) while the gradient's starts from 2(z^L - y)
(Section 3.4); the block-diagonal blocks are the layers (split 1-1-...-1)
unless a split structure is given, in which case the neurons of layer m are
cut into split[m] contiguous groups of near-equal size (group g holds neurons
floor(g n_m / s_m) .. floor((g+1) n_m / s_m) - 1; the paper's example and
Table 2 give only the group counts), a partition is the weights between one
group of layer m-1 and one group of layer m, and b^m_j goes to the partition of
the first group of layer m-1 (Section 3.1); the CG termination rule of
Section 4.4 counts lock-step iterations: the solve ends once CG_min steps are
done and the stated share of partitions have met their own stop rule.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------- layout
def num_params(widths):
    """n = sum_m (n_{m-1} n_m + n_m)  (Section 2.1)."""
    return sum(widths[m - 1] * widths[m] + widths[m] for m in range(1, len(widths)))


def block_slices(widths):
    """Coordinates of layer block m = (w^m, b^m) inside theta, m = 1..L."""
    out, off = [], 0
    for m in range(1, len(widths)):
        size = widths[m - 1] * widths[m] + widths[m]
        out.append(slice(off, off + size))
        off += size
    return out


def unpack(theta, widths):
    """theta -> [(W^m, b^m)], W^m of shape n_{m-1} x n_m.

    w^m lists the columns of W^m one after another (Section 2.1): entry
    w^m_{tj} sits at position j*n_{m-1} + t of the layer's weight run.
    """
    theta = np.asarray(theta, dtype=np.float64)
    layers, off = [], 0
    for m in range(1, len(widths)):
        a, b = widths[m - 1], widths[m]
        W = theta[off:off + a * b].reshape(b, a).T
        off += a * b
        bias = theta[off:off + b]
        off += b
        layers.append((W, bias))
    assert off == theta.size
    return layers


def pack(layers):
    """Inverse of `unpack`."""
    parts = []
    for W, b in layers:
        parts.append(np.asarray(W, dtype=np.float64).T.reshape(-1))
        parts.append(np.asarray(b, dtype=np.float64).reshape(-1))
    return np.concatenate(parts)


# --------------------------------------------------------------------------- forward, f, grad
def sigmoid(s):
    return 1.0 / (1.0 + np.exp(-s))


def forward(theta, widths, X):
    """Eq. (xtoz) with the activation of Section 3.3.2: returns [Z_0, ..., Z_L], rows = instances."""
    layers = unpack(theta, widths)
    L = len(layers)
    Z = [np.asarray(X, dtype=np.float64)]
    for m, (W, b) in enumerate(layers, start=1):
        S = Z[-1] @ W + b
        Z.append(sigmoid(S) if m < L else S)
    return Z


def fun(theta, widths, C, X, Y):
    """Eq. (obj-function) with the squared loss of Eq. (thiswork-loss)."""
    theta = np.asarray(theta, dtype=np.float64)
    ZL = forward(theta, widths, X)[-1]
    l = ZL.shape[0]
    loss = np.sum((ZL - np.asarray(Y, dtype=np.float64)) ** 2)
    return float(theta @ theta / (2.0 * C) + loss / l)


def act_derivative(Z, m, L):
    """sigma'(s^m) = z^m (1 - z^m) below the output layer, 1 at it (Section 3.3.2)."""
    return Z[m] * (1.0 - Z[m]) if m < L else np.ones_like(Z[m])


def backprop(theta, widths, Z, dZL):
    """Eqs. (ztox-g)-(xtow-g-bias) without the 1/C and 1/l factors.

    Given d xi / d z^L for every row, returns sum_i (J^i)^T (dZL row i) in theta layout.
    """
    layers = unpack(theta, widths)
    L = len(layers)
    out = [None] * L
    dZ = dZL
    for m in range(L, 0, -1):
        W, _ = layers[m - 1]
        dS = dZ * act_derivative(Z, m, L)              # (ztox-g)
        gW = Z[m - 1].T @ dS                           # (xtow-g): sum_i z^{m-1}_t dS_j
        gb = dS.sum(axis=0)                            # (xtow-g-bias)
        out[m - 1] = (gW, gb)
        if m > 1:
            dZ = dS @ W.T                              # (communi-g)
    return pack(out)


def grad(theta, widths, C, X, Y):
    """Eq. (whole-gradient); the backward pass starts from 2 (z^L - y) (Section 3.4)."""
    theta = np.asarray(theta, dtype=np.float64)
    Z = forward(theta, widths, X)
    l = Z[0].shape[0]
    dZL = 2.0 * (Z[-1] - np.asarray(Y, dtype=np.float64))
    return theta / C + backprop(theta, widths, Z, dZL) / l


# --------------------------------------------------------------------------- tier D
def jacobian(theta, widths, x):
    """Explicit J^i (n_L x n) for one instance by the backward recurrence of Section 3.3.

    A^m[u, j] = d z^L_u / d z^m_j starts as the identity at m = L (Eq. zLindependent);
    E^m = A^m diag(sigma'(s^m)) is d z^L_u / d s^m_j (Eq. ztox-jaco); the columns of J^i
    for w^m_{tj} are E^m[:, j] z^{m-1}_t and for b^m_j are E^m[:, j] (Eqs. xtow-jaco,
    xtow-jaco-bias); A^{m-1} = E^m (W^m)^T (Eq. communi-jaco).
    """
    layers = unpack(theta, widths)
    L = len(layers)
    Z = forward(theta, widths, np.asarray(x, dtype=np.float64).reshape(1, -1))
    z = [a[0] for a in Z]
    nL = widths[-1]
    J = np.zeros((nL, num_params(widths)))
    blocks = block_slices(widths)
    A = np.eye(nL)
    for m in range(L, 0, -1):
        W, _ = layers[m - 1]
        dsig = z[m] * (1.0 - z[m]) if m < L else np.ones(nL)
        E = A * dsig[None, :]
        a, b = widths[m - 1], widths[m]
        off = blocks[m - 1].start
        for u in range(nL):
            for j in range(b):
                for t in range(a):
                    J[u, off + j * a + t] = E[u, j] * z[m - 1][t]
                J[u, off + a * b + j] = E[u, j]
        A = E @ W.T
    return J


def gauss_newton_dense(theta, widths, C, XS):
    """G^S = I/C + (1/|S|) sum_{i in S} (J^i)^T B^i J^i with B^i = 2I (Eq. sampled-Gauss)."""
    n = num_params(widths)
    G = np.zeros((n, n))
    for x in np.asarray(XS, dtype=np.float64):
        J = jacobian(theta, widths, x)
        G += J.T @ (2.0 * J)
    return np.eye(n) / C + G / len(XS)


def block_diagonal_of(G, widths):
    """Eq. (gausshat): keep the diagonal layer blocks of a dense matrix, zero the rest."""
    H = np.zeros_like(G)
    for sl in block_slices(widths):
        H[sl, sl] = G[sl, sl]
    return H


def Gv_definition(theta, widths, C, XS, v):
    """G^S v accumulated sample by sample from explicit J^i (Eq. real-jaco with one partition)."""
    v = np.asarray(v, dtype=np.float64)
    acc = np.zeros_like(v)
    for x in np.asarray(XS, dtype=np.float64):
        J = jacobian(theta, widths, x)
        acc += J.T @ (2.0 * (J @ v))
    return v / C + acc / len(XS)


def Gv_blockdiag_definition(theta, widths, C, XS, v):
    """Eq. (approx-jaco): each layer block uses only its own columns J^i_p of J^i."""
    v = np.asarray(v, dtype=np.float64)
    acc = np.zeros_like(v)
    blocks = block_slices(widths)
    for x in np.asarray(XS, dtype=np.float64):
        J = jacobian(theta, widths, x)
        for sl in blocks:
            Jp = J[:, sl]
            acc[sl] += Jp.T @ (2.0 * (Jp @ v[sl]))
    return v / C + acc / len(XS)


# --------------------------------------------------------------------------- tier M
def Jv(theta, widths, Z, v):
    """J^i v for every row at once: the directional derivative of Eq. (xtoz) along v.

    With v = (V^1, c^1, ..., V^L, c^L) in theta layout,
    R s^m = R z^{m-1} W^m + z^{m-1} V^m + c^m and R z^m = sigma'(s^m) * R s^m, R z^0 = 0.
    Summing the per-layer terms is the sum over partitions of Eq. (real-jaco).
    """
    layers = unpack(theta, widths)
    dirs = unpack(v, widths)
    L = len(layers)
    RZ = np.zeros_like(Z[0])
    for m in range(1, L + 1):
        W, _ = layers[m - 1]
        V, c = dirs[m - 1]
        RS = RZ @ W + Z[m - 1] @ V + c
        RZ = RS * act_derivative(Z, m, L)
    return RZ


def Gv(theta, widths, C, XS, v):
    """Eq. (sampled-Gauss) applied to v: v/C + (1/|S|) J^T (2 J v)."""
    v = np.asarray(v, dtype=np.float64)
    Z = forward(theta, widths, XS)
    U = 2.0 * Jv(theta, widths, Z, v)                       # B^i = 2I
    return v / C + backprop(theta, widths, Z, U) / Z[0].shape[0]


def Gv_blockdiag(theta, widths, C, XS, v):
    """Eq. (approx-jaco) with one block per layer: block m sees only its own part of v and
    keeps only its own part of J^T (2 J_m v_m)."""
    v = np.asarray(v, dtype=np.float64)
    Z = forward(theta, widths, XS)
    rows = Z[0].shape[0]
    out = v / C
    for sl in block_slices(widths):
        vm = np.zeros_like(v)
        vm[sl] = v[sl]
        U = 2.0 * Jv(theta, widths, Z, vm)
        out[sl] += backprop(theta, widths, Z, U)[sl] / rows
    return out


# --------------------------------------------------------------------------- CG
def cg(matvec, g, lam, max_iter, tol, segments=None, keep_iterates=True):
    """Conjugate gradient on (A + lam I) d = -g, d_0 = 0, no preconditioner.

    Stop rule of Eq. (CG-stopping-cond): ||(A + lam I) d + g|| <= tol ||g|| (the left side
    is the CG residual norm) or `max_iter` steps.  `segments` (list of slices) runs the
    independent systems of Eq. (p-linear) side by side: every scalar is per segment and a
    segment that met its stop rule is frozen.  Returns (d, iterates, resnorms) where
    resnorms[k][s] is segment s's residual norm after k steps (iterates stays empty when
    `keep_iterates` is False: at the largest networks fifty copies of d do not fit).
    """
    g = np.asarray(g, dtype=np.float64)
    if segments is None:
        segments = [slice(0, g.size)]
    d = np.zeros_like(g)
    r = -g.copy()
    p = r.copy()
    rho = np.array([r[s] @ r[s] for s in segments])
    gnorm = np.sqrt(rho.copy())
    active = np.array([tol <= 0 or np.sqrt(rho[k]) > tol * gnorm[k] for k in range(len(segments))])
    active &= rho > 0
    iterates, resnorms = [], [np.sqrt(rho.copy())]
    it = 0
    while it < max_iter and active.any():
        q = matvec(p) + lam * p
        for k, s in enumerate(segments):
            if not active[k]:
                continue
            alpha = rho[k] / (p[s] @ q[s])
            d[s] += alpha * p[s]
            r[s] -= alpha * q[s]
            rho_new = r[s] @ r[s]
            beta = rho_new / rho[k]
            p[s] = r[s] + beta * p[s]
            rho[k] = rho_new
            if tol > 0 and np.sqrt(rho_new) <= tol * gnorm[k]:
                active[k] = False
        it += 1
        if keep_iterates:
            iterates.append(d.copy())
        resnorms.append(np.sqrt(rho.copy()))
    return d, iterates, resnorms


def cg_solve(theta, widths, C, XS, g, lam, blockdiag, max_iter, tol):
    """CG on the full system (Eq. sample-gaussnewton) or the per-layer systems (Eq. block-gaussnewton)."""
    if blockdiag:
        return cg(lambda p: Gv_blockdiag(theta, widths, C, XS, p), g, lam, max_iter, tol,
                  segments=block_slices(widths))
    return cg(lambda p: Gv(theta, widths, C, XS, p), g, lam, max_iter, tol)


# --------------------------------------------------------------------------- variable partition (Section 3.1)
def group_bounds(n, s):
    """Boundaries of the s contiguous neuron groups of a layer with n neurons."""
    return [(g * n) // s for g in range(s + 1)]


def partition_labels(widths, split):
    """Partition id of every coordinate of theta for a split structure split[0..L] (Section 3.1).

    Partitions are numbered layer by layer, and inside layer m by (group of layer m-1, group of layer m) with
    the layer-m group running fastest.  w^m_{tj} belongs to (group of t, group of j); b^m_j to (first group of
    layer m-1, group of j).  Returns (labels, P).
    """
    assert len(split) == len(widths) and all(1 <= s <= n for s, n in zip(split, widths))
    labels = np.empty(num_params(widths), dtype=np.int64)
    off, base = 0, 0
    for m in range(1, len(widths)):
        a, b = widths[m - 1], widths[m]
        ga = np.searchsorted(group_bounds(a, split[m - 1]), np.arange(a), side="right") - 1   # group of neuron t
        gb = np.searchsorted(group_bounds(b, split[m]), np.arange(b), side="right") - 1       # group of neuron j
        lab_w = base + ga[None, :] * split[m] + gb[:, None]          # [j, t], stored with t running fastest
        labels[off:off + a * b] = lab_w.reshape(-1)
        off += a * b
        labels[off:off + b] = base + gb                              # first group of layer m-1
        off += b
        base += split[m - 1] * split[m]
    return labels, base


def partition_indices(widths, split):
    """Index arrays of the P partitions, in partition order."""
    labels, P = partition_labels(widths, split)
    return [np.flatnonzero(labels == p) for p in range(P)]


def partition_diagonal_of(G, widths, split):
    """Eq. (gausshat) for a split structure: keep the entries of a dense matrix whose row and column are in the
    same partition, zero the rest."""
    labels, _ = partition_labels(widths, split)
    return np.where(labels[:, None] == labels[None, :], G, 0.0)


def Gv_partition_definition(theta, widths, C, XS, v, split):
    """Eq. (approx-jaco) from explicit J^i: partition p uses only its own columns J^i_p."""
    v = np.asarray(v, dtype=np.float64)
    parts = partition_indices(widths, split)
    acc = np.zeros_like(v)
    for x in XS:
        J = jacobian(theta, widths, x)
        for idx in parts:
            Jp = J[:, idx]
            acc[idx] += Jp.T @ (2.0 * (Jp @ v[idx]))
    return v / C + acc / len(XS)


def Gv_partition(theta, widths, C, XS, v, split):
    """Eq. (approx-jaco) for a split structure in the order of Section 4.2, all rows at once: for the partition
    (T_{m-1}, T_m), u_i = sum_{t in T_{m-1}} z^{m-1,i}_t mat(v_p)_{t,.} (plus c^m restricted to T_m when
    T_{m-1} is the first group), J_p v_p = D^m_i[:, T_m] u_i (Eq. direct-JV-cost), then
    D^m_i[:, T_m]^T (2 J_p v_p) (Eq. JTv) and the outer product with z^{m-1,i}_{T_{m-1}} (Eq. JTV-independent)."""
    v = np.asarray(v, dtype=np.float64)
    Z = forward(theta, widths, XS)
    D = jacobian_factors(theta, widths, Z)
    dirs = unpack(v, widths)
    rows = Z[0].shape[0]
    out = []
    for m, (V, c) in enumerate(dirs, start=1):
        ba, bb = group_bounds(widths[m - 1], split[m - 1]), group_bounds(widths[m], split[m])
        GW, Gb = np.zeros_like(V), np.zeros_like(c)
        for a in range(split[m - 1]):
            Ta = slice(ba[a], ba[a + 1])
            for b in range(split[m]):
                Tb = slice(bb[b], bb[b + 1])
                U = Z[m - 1][:, Ta] @ V[Ta, Tb]
                if a == 0:
                    U = U + c[Tb]
                Dp = D[m - 1][:, :, Tb]
                P = np.einsum("iuj,ij->iu", Dp, U)
                Q = np.einsum("iuj,iu->ij", Dp, 2.0 * P)
                GW[Ta, Tb] = Z[m - 1][:, Ta].T @ Q / rows
                if a == 0:
                    Gb[Tb] = Q.sum(axis=0) / rows
        out.append((GW, Gb))
    return v / C + pack(out)


def cg_partitioned(theta, widths, C, XS, g, lam, split, max_iter, tol, cg_min=0, finished_share=1.0):
    """The P independent systems of Eq. (p-linear) run in lock step, with the termination rule of Section 4.4:
    every partition stops once at least `cg_min` steps are done and at least `finished_share` of the partitions
    have met Eq. (cg-stopping-sample); a partition that met its own rule earlier stays frozen.
    Returns (d, iterates, resnorms) like `cg`."""
    g = np.asarray(g, dtype=np.float64)
    parts = partition_indices(widths, split)
    P = len(parts)
    d = np.zeros_like(g)
    r = -g.copy()
    p = r.copy()
    rho = np.array([r[s] @ r[s] for s in parts])
    gnorm = np.sqrt(rho.copy())
    active = np.array([tol <= 0 or np.sqrt(rho[k]) > tol * gnorm[k] for k in range(P)]) & (rho > 0)
    iterates, resnorms = [], [np.sqrt(rho.copy())]
    it = 0
    while it < max_iter and active.any():
        if it >= cg_min and (P - active.sum()) >= finished_share * P:
            break
        q = Gv_partition(theta, widths, C, XS, p, split) + lam * p
        for k, s in enumerate(parts):
            if not active[k]:
                continue
            alpha = rho[k] / (p[s] @ q[s])
            d[s] += alpha * p[s]
            r[s] -= alpha * q[s]
            rho_new = r[s] @ r[s]
            p[s] = r[s] + (rho_new / rho[k]) * p[s]
            rho[k] = rho_new
            if tol > 0 and np.sqrt(rho_new) <= tol * gnorm[k]:
                active[k] = False
        it += 1
        iterates.append(d.copy())
        resnorms.append(np.sqrt(rho.copy()))
    return d, iterates, resnorms


# --------------------------------------------------------------------------- Newton iteration (Algorithm 3 on one node)
def combine_directions(a, b, c, r1, r2, eps):
    """Two-variable system of Eq. (sol-comp): [[a, b], [b, c]] (beta1, beta2) = (r1, r2) with
    a = d^T G d, b = dbar^T G d, c = dbar^T G dbar, r1 = -g^T d, r2 = -g^T dbar.
    Eq. (determinant): beta = (1, 0) when the determinant is at most eps."""
    det = a * c - b * b
    if det <= eps:
        return 1.0, 0.0
    return (r1 * c - b * r2) / det, (a * r2 - b * r1) / det


def lm_update(lam, rho, drop, boost):
    """Eq. (LM-rules)."""
    if rho > 0.75:
        return lam * drop
    if rho >= 0.25:
        return lam
    return lam * boost


def newton_iteration(theta, widths, C, X, Y, idx, dprev, lam, sigma=1e-3, eta=1e-4, cg_max=250, eps=1e-5,
                     drop=2.0 / 3.0, boost=1.5, blockdiag=True, max_backtrack=30):
    """One pass of the loop body of Algorithm 3 with a single partition holding everything.

    g on all rows; CG on the (block-diagonal or full) subsampled system with lambda (Eq. block-gaussnewton);
    direction combination with the previous direction on the full G^S (Eq. linear-comb-now); back-tracking
    line search alpha in {1, 1/2, ...} (Eq. linesearch-condition); rho and the next lambda (Eq. LM-rules).
    Returns (theta_next, d, lam_next, report).
    """
    theta = np.asarray(theta, dtype=np.float64)
    dprev = np.asarray(dprev, dtype=np.float64)
    XS = np.asarray(X)[np.asarray(idx)]
    f0 = fun(theta, widths, C, X, Y)
    g = grad(theta, widths, C, X, Y)
    d, its, _ = cg_solve(theta, widths, C, XS, g, lam, blockdiag, cg_max, sigma)
    Gd = Gv(theta, widths, C, XS, d)
    Gdb = Gv(theta, widths, C, XS, dprev)
    a, b, c = d @ Gd, dprev @ Gd, dprev @ Gdb
    beta1, beta2 = combine_directions(a, b, c, -(g @ d), -(g @ dprev), eps)
    dnew = beta1 * d + beta2 * dprev
    gTd = g @ dnew
    dGd = beta1 * beta1 * a + 2.0 * beta1 * beta2 * b + beta2 * beta2 * c
    alpha, backtracks = 1.0, 0
    f1 = fun(theta + alpha * dnew, widths, C, X, Y)
    while f1 > f0 + eta * alpha * gTd and backtracks < max_backtrack:
        alpha *= 0.5
        backtracks += 1
        f1 = fun(theta + alpha * dnew, widths, C, X, Y)
    rho = (f1 - f0) / (alpha * gTd + 0.5 * alpha * alpha * dGd)
    lam_next = lm_update(lam, rho, drop, boost)
    report = dict(f_before=f0, f_after=f1, alpha=alpha, beta1=beta1, beta2=beta2, rho=rho, gTd=gTd, dGd=dGd,
                  cg_iters=len(its), backtracks=backtracks, lambda_next=lam_next)
    return theta + alpha * dnew, dnew, lam_next, report


# --------------------------------------------------------------------------- stored Jacobian factors (Section 3.3.1 / 4.2)
def jacobian_factors(theta, widths, Z):
    """D^m[i, u, j] = d z^{L,i}_u / d s^{m,i}_j for every row i, m = 1..L (Eq. Jelement-store).

    Backward recurrence of Section 3.3 for all rows at once: D^L = I (the output layer is linear),
    D^{m-1} = (D^m W^{mT}) * sigma'(z^{m-1}) (Eq. communi-jaco followed by Eq. ztox-jaco).  Returns [D^1, ..., D^L].
    """
    layers = unpack(theta, widths)
    L = len(layers)
    rows, nL = Z[0].shape[0], widths[-1]
    D = [None] * (L + 1)
    D[L] = np.broadcast_to(np.eye(nL), (rows, nL, nL)).copy()
    for m in range(L, 1, -1):
        W, _ = layers[m - 1]
        D[m - 1] = (D[m] @ W.T) * act_derivative(Z, m - 1, L)[:, None, :]
    return D[1:]


def Gv_blockdiag_stored(theta, widths, C, XS, v):
    """Block-diagonal product the way Section 4.2 orders it: for block m, u_i = V^{mT} z^{m-1,i} + c^m
    (the inner sum of Eq. direct-JV-cost), J_m v_m = D^m_i u_i, then D^{mT}_i (2 J_m v_m) (Eq. JTv), and the
    outer product with z^{m-1,i} summed over rows (Eq. JTV-independent)."""
    v = np.asarray(v, dtype=np.float64)
    Z = forward(theta, widths, XS)
    D = jacobian_factors(theta, widths, Z)
    dirs = unpack(v, widths)
    rows = Z[0].shape[0]
    out = []
    for m, (V, c) in enumerate(dirs, start=1):
        U = Z[m - 1] @ V + c                                  # rows x n_m
        P = np.einsum("iuj,ij->iu", D[m - 1], U)              # J_m v_m per row
        Q = np.einsum("iuj,iu->ij", D[m - 1], 2.0 * P)        # D^T (B J_m v_m), B = 2I
        out.append((Z[m - 1].T @ Q / rows, Q.sum(axis=0) / rows))
    return v / C + pack(out)
