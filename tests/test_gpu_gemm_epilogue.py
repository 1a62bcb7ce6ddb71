"""Epilogue options of the contraction kernels, one kernel at a time and in every combination:
D = alpha * dsig'(f(A B + 1 bias^T)) + beta * cin (Eqs. xtoz, ztox-g, xtow-g with the regulariser as the accumulate
term), against the same expression in float64 numpy.  The path uses one option at a time; the kernels compile a
form per option and a run-time form for combinations, and this file puts all of them through each kernel."""
import itertools

import numpy as np
import pytest

import gn_workloads as wl

pytestmark = pytest.mark.gpu

# (M, N, K): several tiles with a ragged last tile and a ragged last 32-column chunk; one tile exactly; more rows
# than one wave of CTA pairs covers, so that tiles are also cut along K (kind 5)
SHAPES = [(700, 520, 264), (256, 256, 96), (19200, 264, 2016)]
# kind -> (relative L2 bound, needs operands with slack behind them)
KINDS = {1: (2e-6, False), 4: (2e-3, True), 5: (2e-3, True), 6: (2e-3, True), 7: (4e-6, False)}
COMBOS = [c for c in itertools.product((0, 1), repeat=4)]     # (bias, sigmoid, dsig, cin)


@pytest.fixture(scope="module")
def ctx():
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make("tiny")
    c = gn.GnContext(p["widths"], p["C"], torch.from_numpy(p["X"]).cuda(), torch.from_numpy(p["Y"]).cuda())
    yield c
    c.close()


def reference(A, B, a_k, b_k, bias, sigmoid, z, alpha, cin, beta):
    Am = A if a_k else A.T
    Bm = B.T if b_k else B
    x = Am.astype(np.float64) @ Bm.astype(np.float64)
    if bias is not None:
        x = x + bias.astype(np.float64)[None, :]
    if sigmoid:
        x = 1.0 / (1.0 + np.exp(-x))
    if z is not None:
        zz = z.astype(np.float64)
        x = x * zz * (1.0 - zz)
    x = alpha * x
    if cin is not None:
        x = x + beta * cin.astype(np.float64)
    return x


def slack(t):
    import torch
    buf = torch.zeros(t.size + 64, dtype=torch.float32, device="cuda")
    return buf[: t.size].view(t.shape).copy_(torch.from_numpy(t))


@pytest.mark.parametrize("a_k,b_k", [(True, True), (False, False), (True, False)])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("kind", sorted(KINDS))
def test_every_combination_of_epilogue_options(ctx, kind, shape, a_k, b_k):
    import torch
    M, N, K = shape
    if kind == 1 and M > 5000:
        pytest.skip("the FP32 FMA kernel has no K slices to exercise")
    tol, need_slack = KINDS[kind]
    rng = np.random.Generator(np.random.PCG64(1000 * kind + M + 3 * N + 7 * K))
    A = (0.5 * rng.standard_normal((M, K) if a_k else (K, M))).astype(np.float32)
    B = (0.5 * rng.standard_normal((N, K) if b_k else (K, N))).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    z = rng.uniform(0.05, 0.95, size=(M, N)).astype(np.float32)
    cin = rng.standard_normal((M, N)).astype(np.float32)
    up = slack if need_slack else (lambda t: torch.from_numpy(t).cuda())
    dA, dB = up(A), up(B)
    dbias, dz, dcin = torch.from_numpy(bias).cuda(), torch.from_numpy(z).cuda(), torch.from_numpy(cin).cuda()
    for use_bias, sigmoid, use_dsig, use_cin in COMBOS:
        alpha, beta = (0.75, -1.5) if use_cin else (2.0, 0.0)
        D = ctx.debug_gemm_epilogue(kind, dA, dB, a_kmajor=a_k, b_kmajor=b_k, bias=dbias if use_bias else None,
                                    sigmoid=bool(sigmoid), dsig=dz if use_dsig else None, alpha=alpha,
                                    cin=dcin if use_cin else None, beta=beta).cpu().numpy().astype(np.float64)
        ref = reference(A, B, a_k, b_k, bias if use_bias else None, sigmoid, z if use_dsig else None, alpha,
                        cin if use_cin else None, beta)
        err = np.linalg.norm(D - ref) / np.linalg.norm(ref)
        assert err <= tol, (kind, shape, (use_bias, sigmoid, use_dsig, use_cin), err)
        # and element by element: no chunk, row or tile may be off while the norm hides it
        scale = np.abs(ref).max()
        assert np.abs(D - ref).max() <= 50 * tol * scale, (kind, shape, (use_bias, sigmoid, use_dsig, use_cin))


@pytest.mark.parametrize("shape,a_k,b_k", [((3000, 520, 12), True, False),      # thin-K: K <= 16
                                            ((12, 520, 3000), False, False),     # thin-M: M <= 16
                                            ((3000, 12, 520), True, True)])      # thin-N: N <= 16
def test_streaming_kernels_with_every_combination(ctx, shape, a_k, b_k):
    import torch
    M, N, K = shape
    rng = np.random.Generator(np.random.PCG64(M + 3 * N + 7 * K))
    A = (0.5 * rng.standard_normal((M, K) if a_k else (K, M))).astype(np.float32)
    B = (0.5 * rng.standard_normal((N, K) if b_k else (K, N))).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    z = rng.uniform(0.05, 0.95, size=(M, N)).astype(np.float32)
    cin = rng.standard_normal((M, N)).astype(np.float32)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    dbias, dz, dcin = torch.from_numpy(bias).cuda(), torch.from_numpy(z).cuda(), torch.from_numpy(cin).cuda()
    for use_bias, sigmoid, use_dsig, use_cin in COMBOS:
        alpha, beta = (0.75, -1.5) if use_cin else (2.0, 0.0)
        D = ctx.debug_gemm_epilogue(2, dA, dB, a_kmajor=a_k, b_kmajor=b_k, bias=dbias if use_bias else None,
                                    sigmoid=bool(sigmoid), dsig=dz if use_dsig else None, alpha=alpha,
                                    cin=dcin if use_cin else None, beta=beta).cpu().numpy().astype(np.float64)
        ref = reference(A, B, a_k, b_k, bias if use_bias else None, sigmoid, z if use_dsig else None, alpha,
                        cin if use_cin else None, beta)
        err = np.linalg.norm(D - ref) / np.linalg.norm(ref)
        assert err <= 2e-6, (shape, (use_bias, sigmoid, use_dsig, use_cin), err)
