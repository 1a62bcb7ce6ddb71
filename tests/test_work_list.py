"""Host logic of the grouped / chained launches of the CTA-pair kernel: the work list (no GPU needed)."""
import numpy as np
import pytest

import paper_1802_00130_b200 as gn

PAIRS = 74
COST = lambda kb, bn: kb * (256.0 + bn) / 512.0 + 8.0     # the library's tile-time model, restated


def kblocks(K):
    return (K + 31) // 32


CASES = [
    [(2000, 2000, 12000), (12000, 2000, 2000)],                       # weight block + activation gradient, |S| = 12000
    [(2000, 2000, 3000), (3000, 2000, 2000)],                         # the same at |S| = 3000
    [(12000, 2000, 784), (12000, 2000, 2000), (12000, 2000, 2000)],   # stage 1 of the stored-factor product
    [(2000, 784, 12000), (2000, 2000, 12000), (2000, 2000, 12000)],   # its stage 3
    [(300, 520, 1100), (1100, 392, 520)],                             # ragged sizes, fewer tiles than pairs
    [(4096, 4096, 20000), (20000, 4096, 4096)],
    [(32768, 2000, 784), (32768, 2000, 2000), (32768, 2000, 2000), (32768, 2000, 2000), (32768, 256, 2000)],
]


@pytest.mark.parametrize("keep_order", [False, True])
@pytest.mark.parametrize("shapes", CASES)
def test_every_tile_is_dealt_once_and_the_loads_come_out_even(shapes, keep_order):
    used, order, tiles, waves, counts = gn.plan_group(shapes, PAIRS, keep_order)
    n = len(shapes)
    assert sorted(order) == list(range(n))
    if keep_order:
        assert order == list(range(n))
    load = np.zeros(PAIRS)
    costs = []
    for k in range(n):
        M, N, K = shapes[order[k]]
        tiles_m = (M + 255) // 256
        assert tiles[k] % tiles_m == 0                        # whole rows of tiles
        bn = -(-N // (tiles[k] // tiles_m))                   # (the width is not reported: bound it from the count)
        assert sum(counts[k]) == tiles[k]                     # every tile exactly once
        assert all(c >= waves[k] for c in counts[k][:used]) and all(c == 0 for c in counts[k][used:])
        assert min(counts[k][:used]) == waves[k]              # the whole waves are all the waves every pair runs
        cost = COST(kblocks(K), min(256, max(128, -(-bn // 64) * 64)))
        costs.append(cost)
        load += np.array(counts[k]) * cost
    if not keep_order:
        # longest tiles first
        per_tile = [costs[k] for k in range(n)]
        assert per_tile == sorted(per_tile, reverse=True)
    # as even as whole tiles allow: no pair carries more than the mean plus one of the largest tiles
    assert load[:used].max() <= load[:used].mean() + max(costs) + 1e-9
    assert used == min(PAIRS, sum(tiles))


def test_bad_arguments_are_refused():
    with pytest.raises(ValueError):
        gn.plan_group([(0, 10, 10)])
    with pytest.raises(ValueError):
        gn.plan_group([(256, 256, 256)] * 7)                 # more problems than a launch takes
    with pytest.raises(ValueError):
        gn.plan_group([(256, 256, 256)], pairs=81)
