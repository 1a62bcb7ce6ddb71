"""Pins for the oracle's variable-partition functions (Sections 3.1, 4.1, 4.2, 4.4): counts the paper prints,
the dense matrix with cross-partition entries zeroed, and special cases that reduce to functions pinned elsewhere."""
import os

import numpy as np
import pytest

import gn_workloads as wl
from oracle import gn_oracle as orc


def rel(a, b):
    return float(np.linalg.norm(np.asarray(a) - np.asarray(b)) / np.linalg.norm(b))


def small(widths, rows=7, seed=5):
    rng = np.random.Generator(np.random.PCG64(seed))
    n = orc.num_params(widths)
    theta = rng.standard_normal(n) * 0.7
    X = rng.standard_normal((rows, widths[0]))
    v = rng.standard_normal(n)
    return theta, X, v


def test_partition_counts_printed_in_the_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "partition_counts.txt")
    seen = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        net, split, count = line.split()
        widths = [int(x) for x in net.split("-")]
        s = [int(x) for x in split.split("-")]
        labels, P = orc.partition_labels(widths, s)
        assert P == int(count), line
        assert set(labels.tolist()) == set(range(P))            # every partition is non-empty, every variable has one
        seen += 1
    assert seen == 10


def test_worked_example_of_the_variable_partition():
    # 150-200-30 split 3-2-3 (Section 3.1): (A_0, A_1) owns a 50 x 100 block of W^1 and 100 biases of b^1
    widths, split = [150, 200, 30], [3, 2, 3]
    labels, P = orc.partition_labels(widths, split)
    parts = orc.partition_indices(widths, split)
    assert P == 12 and len(parts[0]) == 50 * 100 + 100 and len(parts[1]) == 50 * 100 + 100
    # the other first-layer partitions hold weights only
    for p in range(2, 6):
        assert len(parts[p]) == 50 * 100
    # b^1 (coordinates 30000..30199) is split 100 / 100 between (A_0, A_1) and (A_0, B_1)
    b1 = labels[150 * 200:150 * 200 + 200]
    assert (b1[:100] == 0).all() and (b1[100:] == 1).all()
    # w^1_{tj} with t = 60 (group B_0), j = 150 (group B_1) sits at j * 150 + t
    assert labels[150 * 150 + 60] == 1 * 2 + 1
    # second layer: 2 x 3 partitions of 100 x 10 weights, biases with the first group of layer 1
    assert sorted(len(x) for x in parts[6:]) == [1000, 1000, 1000, 1010, 1010, 1010]
    assert sum(len(x) for x in parts) == orc.num_params(widths)


@pytest.mark.parametrize("widths,split", [([5, 6, 4, 3], [2, 3, 2, 1]), ([4, 7, 3], [1, 2, 3]), ([6, 5], [3, 2]),
                                          ([5, 4, 4, 2], [1, 1, 1, 1])])
def test_partition_product_is_the_dense_matrix_with_cross_partition_entries_zeroed(widths, split):
    theta, X, v = small(widths)
    C = 3.0
    G = orc.gauss_newton_dense(theta, widths, C, X)
    ref = orc.partition_diagonal_of(G, widths, split) @ v
    assert rel(orc.Gv_partition_definition(theta, widths, C, X, v, split), ref) <= 1e-12
    assert rel(orc.Gv_partition(theta, widths, C, X, v, split), ref) <= 1e-12


def test_unit_split_is_the_layer_block_product_and_finer_splits_differ():
    widths = [6, 8, 5, 3]
    theta, X, v = small(widths)
    ones = [1] * len(widths)
    a = orc.Gv_partition(theta, widths, 2.0, X, v, ones)
    assert rel(a, orc.Gv_blockdiag(theta, widths, 2.0, X, v)) <= 1e-12
    assert rel(a, orc.Gv_blockdiag_stored(theta, widths, 2.0, X, v)) <= 1e-12
    b = orc.Gv_partition(theta, widths, 2.0, X, v, [2, 2, 1, 1])
    assert rel(b, a) > 1e-3                                      # dropping cross-group terms changes the product


def test_direction_supported_on_one_partition_sees_the_full_matrix_there():
    widths, split = [6, 8, 5, 3], [2, 2, 2, 1]
    theta, X, v = small(widths)
    parts = orc.partition_indices(widths, split)
    for p in (0, 3, 5, len(parts) - 1):
        vp = np.zeros_like(v)
        vp[parts[p]] = v[parts[p]]
        full = orc.Gv(theta, widths, 4.0, X, vp)
        hat = orc.Gv_partition(theta, widths, 4.0, X, vp, split)
        assert rel(hat[parts[p]], full[parts[p]]) <= 1e-12
        rest = np.setdiff1d(np.arange(v.size), parts[p])
        assert np.abs(hat[rest]).max() == 0.0                    # v / C and the product vanish off the partition


def test_partition_product_is_symmetric_and_bounded_below():
    widths, split = [7, 9, 6, 4], [3, 2, 3, 2]
    theta, X, v = small(widths)
    u = small(widths, seed=9)[2]
    C = 5.0
    Gu, Gv_ = (orc.Gv_partition(theta, widths, C, X, w, split) for w in (u, v))
    assert abs(u @ Gv_ - v @ Gu) <= 1e-12 * abs(u @ Gv_)
    assert v @ Gv_ >= v @ v / C


def test_partitioned_cg_solves_every_partition_system():
    widths, split = [4, 5, 3], [2, 2, 1]
    theta, X, _ = small(widths, rows=9)
    rng = np.random.Generator(np.random.PCG64(3))
    g = rng.standard_normal(orc.num_params(widths))
    C, lam = 2.0, 0.5
    Ghat = orc.partition_diagonal_of(orc.gauss_newton_dense(theta, widths, C, X), widths, split)
    parts = orc.partition_indices(widths, split)
    d, its, res = orc.cg_partitioned(theta, widths, C, X, g, lam, split, max_iter=40, tol=1e-13)
    for idx in parts:
        A = Ghat[np.ix_(idx, idx)] + lam * np.eye(len(idx))
        assert rel(d[idx], np.linalg.solve(A, -g[idx])) <= 1e-9
    # unit split: the same iterates as the per-layer solver pinned elsewhere
    d1, it1, _ = orc.cg_partitioned(theta, widths, C, X, g, lam, [1, 1, 1], max_iter=6, tol=0.0)
    d2, it2, _ = orc.cg_solve(theta, widths, C, X, g, lam, True, 6, 0.0)
    for a, b in zip(it1, it2):
        assert rel(a, b) <= 1e-12


def test_termination_rule_of_the_synchronisation_section():
    widths, split = [10, 9, 6, 3], [2, 3, 2, 1]               # 14 partitions that finish after 2, 3 or 4 steps
    theta, X, _ = small(widths, rows=40)
    rng = np.random.Generator(np.random.PCG64(4))
    g = rng.standard_normal(orc.num_params(widths))
    tol, lam = 1e-3, 0.05
    _, its_all, res_all = orc.cg_partitioned(theta, widths, 2.0, X, g, lam, split, 60, tol)
    n_all = len(its_all)
    res_all = np.array(res_all)
    g0 = res_all[0]
    done_at = [(res_all[:, k] <= tol * g0[k]).argmax() for k in range(res_all.shape[1])]   # first step each one is done
    assert n_all == max(done_at)                              # share 1.0: the slowest partition decides
    assert len(set(done_at)) >= 3
    # 40 % of the partitions finished: stops at the step the 6th of 14 finishes, but not before cg_min
    k_share = sorted(done_at)[5]
    _, its_half, _ = orc.cg_partitioned(theta, widths, 2.0, X, g, lam, split, 60, tol, cg_min=0, finished_share=0.4)
    assert len(its_half) == k_share < n_all
    _, its_min, _ = orc.cg_partitioned(theta, widths, 2.0, X, g, lam, split, 60, tol, cg_min=k_share + 1,
                                       finished_share=0.4)
    assert len(its_min) == k_share + 1 < n_all
    # the iterates up to the early stop are those of the full run
    for a, b in zip(its_half, its_all):
        assert rel(a, b) <= 1e-14
