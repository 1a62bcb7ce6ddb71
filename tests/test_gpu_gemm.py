"""The two contraction kernels on their own, against a float64 matrix product (numpy)."""
import numpy as np
import pytest

import gn_workloads as wl

pytestmark = pytest.mark.gpu

SHAPES = [(128, 256, 32), (128, 256, 64), (300, 520, 200), (1000, 300, 784), (37, 40, 12), (2500, 1000, 1000),
          (260, 2000, 3000), (3000, 10, 2000), (1000, 24, 520), (12000, 2000, 784), (2000, 784, 3000), (19000, 520, 200)]


@pytest.fixture(scope="module")
def ctx():
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make("tiny")
    X = torch.from_numpy(p["X"]).cuda()
    Y = torch.from_numpy(p["Y"]).cuda()
    c = gn.GnContext(p["widths"], p["C"], X, Y)
    yield c
    c.close()


def operands(M, N, K, a_k, b_k, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    A = rng.standard_normal((M, K) if a_k else (K, M), dtype=np.float32)
    B = rng.standard_normal((N, K) if b_k else (K, N), dtype=np.float32)
    Am = A if a_k else A.T
    Bm = B.T if b_k else B
    ref = Am.astype(np.float64) @ Bm.astype(np.float64)
    return A, B, ref


@pytest.mark.parametrize("a_k,b_k", [(True, True), (True, False), (False, True), (False, False)])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("kind,tol", [(1, 2e-6), (0, 1e-3), (3, 1e-3), (4, 1e-3), (5, 1e-3), (6, 1e-3), (7, 2e-6)])
def test_gemm_layouts(ctx, kind, tol, shape, a_k, b_k):
    import torch
    import paper_1802_00130_b200 as gn
    M, N, K = shape
    A, B, ref = operands(M, N, K, a_k, b_k, seed=M + 7 * N + 13 * K)
    if 3 <= kind <= 6:      # operands with readable slack after their last row, as the library's own workspaces have
        bufA = torch.zeros(A.size + 64, dtype=torch.float32, device="cuda")
        bufB = torch.zeros(B.size + 64, dtype=torch.float32, device="cuda")
        dA = bufA[: A.size].view(A.shape).copy_(torch.from_numpy(A))
        dB = bufB[: B.size].view(B.shape).copy_(torch.from_numpy(B))
    else:
        dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    try:
        D = ctx.debug_gemm(kind, dA, dB, a_kmajor=a_k, b_kmajor=b_k)
    except gn.GnError as e:
        if kind == 7:   # the error-compensated form serves the shapes of the CTA-pair kernel only (any alignment)
            assert e.status == 1 and (M <= 128 or N < 128)
            return
        # the tensor-core kernel refuses operands TMA cannot address (leading dimension not a multiple of 4)
        assert kind in (0, 3, 4, 5, 6) and e.status == 1
        lda, ldb = A.shape[1], B.shape[1]
        assert lda % 4 or ldb % 4 or N < 32
        return
    err = np.linalg.norm(D.cpu().numpy() - ref) / np.linalg.norm(ref)
    assert err <= tol, err
    # element-wise too: a misplaced tile would hide in a norm of a large matrix
    assert np.max(np.abs(D.cpu().numpy() - ref)) <= 50 * tol * np.sqrt(K)


THIN = [  # (M, N, K, a_kmajor, b_kmajor): one dimension <= 16, as at the n_L-wide output layer
    (3000, 10, 2000, True, True), (131, 4, 64, True, True), (1000, 16, 300, True, True),
    (10, 2000, 3000, False, False), (4, 16, 131, False, False), (16, 300, 70000, False, False),
    (3000, 2000, 10, True, False), (131, 16, 4, True, False), (777, 300, 16, True, False),
]


@pytest.mark.parametrize("M,N,K,a_k,b_k", THIN)
def test_streaming_kernels_for_thin_shapes(ctx, M, N, K, a_k, b_k):
    import torch
    A, B, ref = operands(M, N, K, a_k, b_k, seed=M + 7 * N + 13 * K)
    D = ctx.debug_gemm(2, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), a_kmajor=a_k, b_kmajor=b_k)
    err = np.linalg.norm(D.cpu().numpy() - ref) / np.linalg.norm(ref)
    assert err <= 2e-6, err
    assert np.max(np.abs(D.cpu().numpy() - ref)) <= 1e-4 * np.sqrt(K)


def test_error_compensated_form_at_long_k_with_one_signed_terms(ctx):
    """All products positive and K = 40000: the worst case for an accumulator that truncates.  The chunked
    accumulation must keep the result within 2e-6 of float64 with no drift towards zero worth speaking of."""
    import torch
    rng = np.random.Generator(np.random.PCG64(77))
    M, N, K = 256, 256, 40000
    A = rng.uniform(0.05, 1.0, (K, M)).astype(np.float32)          # [K][M] and [K][N]: the weight-block layout
    B = rng.uniform(0.05, 1.0, (K, N)).astype(np.float32)
    ref = A.astype(np.float64).T @ B.astype(np.float64)
    D = ctx.debug_gemm(7, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), a_kmajor=False, b_kmajor=False)
    D = D.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(D - ref) / np.linalg.norm(ref) <= 2e-6
    assert abs(np.mean(D - ref)) / np.mean(ref) <= 1.5e-6
