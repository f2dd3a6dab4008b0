"""Pins of the oracle's cube order and of the selection with the own block forced in.

The paper defines both only in the caption of its overview figure (tokens grouped into local 3D
cubes; attention in the own cube beside the top-k selection of cubes); the pins are what the
wording and the arithmetic fix: a hand-worked grid, the properties of a cube, brute force."""
import itertools

import numpy as np

from oracle import usv_oracle as oracle


def test_hand_worked_grid():
    # grid 1 x 2 x 3, cubes 1 x 2 x 2: the first cube holds columns 0-1 of both rows (raster
    # 0,1,3,4), the second, cut by the edge, column 2 (raster 2,5)
    perm, inv = oracle.cube_order((1, 2, 3), (1, 2, 2))
    assert perm.tolist() == [0, 1, 3, 4, 2, 5]
    assert inv.tolist() == [0, 1, 4, 2, 3, 5]


def test_against_nested_loops():
    for grid, cube in [((5, 6, 7), (4, 4, 4)), ((3, 9, 10), (2, 4, 3)), ((8, 8, 8), (4, 4, 4))]:
        T, Hh, W = grid
        ct, ch, cw = cube
        order = []
        for tc, yc, xc in itertools.product(range(-(-T // ct)), range(-(-Hh // ch)), range(-(-W // cw))):
            for lt, ly, lx in itertools.product(range(ct), range(ch), range(cw)):
                t, y, x = tc * ct + lt, yc * ch + ly, xc * cw + lx
                if t < T and y < Hh and x < W:
                    order.append((t * Hh + y) * W + x)
        perm, inv = oracle.cube_order(grid, cube)
        assert perm.tolist() == order
        assert sorted(order) == list(range(T * Hh * W))
        assert np.array_equal(perm[inv], np.arange(T * Hh * W))


def test_whole_cubes_are_64_token_blocks():
    # grid a multiple of the 4 x 4 x 4 cube: every run of 64 positions is exactly one cube
    grid = (8, 12, 16)
    perm, _ = oracle.cube_order(grid, (4, 4, 4))
    t, rem = np.divmod(perm, grid[1] * grid[2])
    y, x = np.divmod(rem, grid[2])
    for blk in range(perm.size // 64):
        s = slice(64 * blk, 64 * blk + 64)
        for c in (t[s], y[s], x[s]):
            assert c.max() - c.min() == 3 and c.min() % 4 == 0


def test_degenerate_cubes_leave_the_raster_order():
    n = 3 * 5 * 7
    assert oracle.cube_order((3, 5, 7), (1, 1, 7))[0].tolist() == list(range(n))
    assert oracle.cube_order((3, 5, 7), (3, 5, 7))[0].tolist() == list(range(n))
    assert oracle.cube_order((3, 5, 7), (1, 1, 1))[0].tolist() == list(range(n))


def test_local_selection_brute_force():
    rng = np.random.default_rng(11)
    s = rng.standard_normal((1, 2, 6, 6))
    s[0, 0, 2, :] = 0.25                      # a constant row: ties go to the lowest index
    kph = [3, 1]
    sel, gap = oracle.select_blocks_local(s, kph)
    for h, k in enumerate(kph):
        for i in range(6):
            best = None
            for sub in itertools.combinations(range(6), k):
                if i not in sub:
                    continue
                key = (-sum(s[0, h, i, j] for j in sub), sub)   # largest total, then lowest indices
                if best is None or key < best:
                    best = key
            assert sel[0, h, i, :k].tolist() == list(best[1])
            assert np.all(sel[0, h, i, k:] == -1)
    assert sel[0, 0, 2, :3].tolist() == [0, 1, 2]
    assert np.all(sel[0, 1, :, 0] == np.arange(6))              # k = 1: the own block alone


def test_local_selection_differs_from_plain_only_by_the_own_block():
    rng = np.random.default_rng(5)
    s = rng.standard_normal((1, 1, 16, 16))
    k = [4]
    plain, _ = oracle.select_blocks(s, k)
    local, _ = oracle.select_blocks_local(s, k)
    for i in range(16):
        p, l = set(plain[0, 0, i].tolist()), set(local[0, 0, i].tolist())
        assert i in l
        if i in p:
            assert p == l
        else:
            # the own block replaces the weakest of the plain choice
            weakest = min(p, key=lambda j: (s[0, 0, i, j], -j))
            assert l == (p - {weakest}) | {i}
