"""Pins of the CPU oracle's token merge / unmerge (Sec. 3.3) against brute force, invariants,
special cases and a hand-derived example."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


def _f64(x):
    return x.to(torch.float64).numpy()


GRID, PART = (3, 4, 6), (1, 1, 2)          # 72 tokens, even raster indices are destinations


def test_destination_mask_counts_and_positions():
    m = oracle.destination_mask(GRID, PART)
    assert m.sum() == 36 and np.array_equal(np.nonzero(m)[0], np.arange(0, 72, 2))
    # general partition with ragged edges: one destination per (cut) block, at its first token
    T, Hh, W, st, sh, sw = 5, 5, 7, 2, 2, 3
    m = oracle.destination_mask((T, Hh, W), (st, sh, sw)).reshape(T, Hh, W)
    assert m.sum() == -(-T // st) * -(-Hh // sh) * -(-W // sw)
    ref = np.zeros_like(m)
    ref[::st, ::sh, ::sw] = True
    assert np.array_equal(m, ref)


def test_descriptors_and_matching_against_numpy_brute_force():
    B, N, Hm, dm = 2, 72, 3, 8
    metric = _rand_bf16((B, N, Hm, dm), 1)
    mhat = oracle.merge_descriptors(metric)
    m = _f64(metric).mean(2)
    ref_hat = m / np.linalg.norm(m, axis=-1, keepdims=True)
    assert np.allclose(mhat, ref_hat, rtol=1e-13, atol=1e-15)
    sl, js, u, u2 = oracle.merge_match(mhat, GRID, PART)
    dst = np.arange(0, N, 2)
    src = np.arange(1, N, 2)
    assert np.array_equal(sl[:, 1], np.tile(src, B))
    for b in range(B):
        cos = ref_hat[b][src] @ ref_hat[b][dst].T          # sources x destinations
        assert cos.min() >= -1 - 1e-12 and cos.max() <= 1 + 1e-12
        s = slice(b * src.size, (b + 1) * src.size)
        assert np.array_equal(js[s], dst[cos.argmax(1)])
        assert np.allclose(u[s], cos.max(1), rtol=1e-13)
        assert np.allclose(u2[s], np.sort(cos, 1)[:, -2], rtol=1e-13)
    # matching never crosses batch elements: changing element 1 leaves element 0 untouched
    metric2 = metric.clone()
    metric2[1] = _rand_bf16((N, Hm, dm), 99)
    _, js2, _, _ = oracle.merge_match(oracle.merge_descriptors(metric2), GRID, PART)
    assert np.array_equal(js2[:src.size], js[:src.size])


def test_match_ties_go_to_lowest_destination_and_duplicates_score_one():
    N, dm = 72, 4
    metric = _rand_bf16((1, N, 1, dm), 2)
    metric[0, 10] = metric[0, 30]            # two identical destinations
    metric[0, 11] = metric[0, 30]            # a source equal to both
    plan = oracle.merge_plan(metric, GRID, PART, r=36)
    assert plan["jstar"][0, 11] == 10        # lowest index among the tied best
    assert abs(plan["u"][0, 11] - 1.0) < 1e-15
    assert abs(plan["u2"][0, 11] - 1.0) < 1e-15
    # a zero descriptor has cosine 0 with everything and so picks destination 0
    metric[0, 13] = 0
    plan = oracle.merge_plan(metric, GRID, PART, r=36)
    assert plan["u"][0, 13] == 0.0 and plan["jstar"][0, 13] == 0


@pytest.mark.parametrize("r", [0, 1, 7, 35, 36])
def test_plan_invariants(r):
    B, N = 2, 72
    metric = _rand_bf16((B, N, 2, 8), 3)
    plan = oracle.merge_plan(metric, GRID, PART, r)
    is_dst = oracle.destination_mask(GRID, PART)
    dst_of, pos, Nm = plan["dst_of"], plan["pos"], plan["Nm"]
    assert Nm == N - r
    for b in range(B):
        merged = dst_of[b] >= 0
        assert merged.sum() == r and not np.any(merged & is_dst)
        assert np.all(is_dst[dst_of[b][merged]])                       # j* is a destination
        assert np.array_equal(dst_of[b][merged], plan["jstar"][b][merged])
        unm = ~merged & ~is_dst
        # merged order: unmerged sources ascending, then destinations ascending
        assert np.array_equal(pos[b][unm], np.arange(unm.sum()))
        assert np.array_equal(pos[b][is_dst], unm.sum() + np.arange(is_dst.sum()))
        assert np.array_equal(pos[b][merged], pos[b][dst_of[b][merged]])
        # group sizes add up to N
        counts = np.bincount(pos[b], minlength=Nm)
        assert counts.sum() == N and counts.min() >= 1 and np.all(counts[:unm.sum()] == 1)
        # the r merged sources are the r most confident ones
        u = plan["u"][b]
        if 0 < r < 36:
            assert u[merged].min() >= u[unm].max()
            assert np.isclose(plan["theta"][b, 0], u[merged].min())
            assert np.isclose(plan["theta"][b, 1], u[unm].max())
    if r == 36:
        assert np.all(pos[:, is_dst] == np.arange(36))                 # U is empty


def test_top_r_ties_go_to_lowest_source_index():
    src = np.arange(1, 21, 2).astype(np.int32)
    u = np.array([.5, .9, .5, .5, .1, .9, .5, .2, .5, .3])
    merged, theta = oracle.merge_select(src, u, 4)
    assert np.array_equal(np.nonzero(merged)[0], [0, 1, 2, 5])        # two .9s, first two .5s
    assert theta[0] == .5 and theta[1] == .5


def test_merge_zero_is_identity_and_merge_values_are_group_means():
    B, N, C = 2, 72, 16
    x = _rand_bf16((B, N, C), 4)
    metric = _rand_bf16((B, N, 2, 8), 5)
    plan0 = oracle.merge_plan(metric, GRID, PART, 0)
    is_dst = oracle.destination_mask(GRID, PART)
    order = np.concatenate([np.nonzero(~is_dst)[0], np.nonzero(is_dst)[0]])
    y0 = oracle.merge_apply(x, plan0["dst_of"], plan0["pos"], plan0["Nm"])
    assert np.array_equal(y0, _f64(x)[:, order])                        # a pure reordering
    back = oracle.unmerge(oracle.round_to_bf16(y0), plan0["pos"])
    assert np.array_equal(back, oracle.bf16_bits(x))                    # unmerge(merge) = id
    # r > 0: every merged row is the plain mean of the tokens that map to it
    plan = oracle.merge_plan(metric, GRID, PART, 20)
    y = oracle.merge_apply(x, plan["dst_of"], plan["pos"], plan["Nm"])
    xf = _f64(x)
    for b in range(B):
        for row in range(plan["Nm"]):
            members = np.nonzero(plan["pos"][b] == row)[0]
            assert np.allclose(y[b, row], xf[b, members].mean(0), rtol=1e-13, atol=1e-15)
            non_merged = [m for m in members if plan["dst_of"][b, m] < 0]
            assert len(non_merged) == 1                                 # exactly one owner


def test_merge_unmerge_merge_is_merge_and_duplicate_roundtrip():
    B, N, C = 1, 72, 8
    metric = _rand_bf16((B, N, 2, 8), 6)
    x = _rand_bf16((B, N, C), 7)
    plan = oracle.merge_plan(metric, GRID, PART, 25)
    args = (plan["dst_of"], plan["pos"], plan["Nm"])
    y = oracle.round_to_bf16(oracle.merge_apply(x, *args))
    xr = oracle.unmerge(y, plan["pos"])
    y2 = oracle.merge_apply(xr, *args)
    assert np.array_equal(oracle.round_to_bf16(y2), y)      # mean of equal copies = the copy
    # if every merged source duplicates its destination's features, the round trip is exact
    xd = x.clone()
    for n in np.nonzero(plan["dst_of"][0] >= 0)[0]:
        xd[0, n] = xd[0, plan["dst_of"][0, n]]
    yd = oracle.round_to_bf16(oracle.merge_apply(xd, *args))
    assert np.array_equal(oracle.unmerge(yd, plan["pos"]), oracle.bf16_bits(xd))


def test_hand_worked_merge_example():
    """1 x 1 x 6 grid, partition (1,1,2): destinations 0,2,4; sources 1,3,5.  Descriptors are
    plane vectors at hand-picked angles; expected plan and merged values are derived in
    tests/golden/merge_hand_example.txt."""
    path = os.path.join(GOLDEN, "merge_hand_example.txt")
    vals = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            key, *rest = line.split()
            vals[key] = [float(t) for t in rest]
    # unit vectors with exactly representable coordinates (3-4-5 and axis directions)
    desc = {0: (1, 0), 2: (0, 1), 4: (-1, 0), 1: (0.75, 1.0), 3: (1.0, 0.125), 5: (-0.5, -0.5)}
    metric = torch.zeros(1, 6, 2, 2)
    for n, (a, b) in desc.items():
        metric[0, n, 0] = torch.tensor([a, b]) * 2   # two heads whose mean is (a, b) * 1.5
        metric[0, n, 1] = torch.tensor([a, b])
    x = torch.arange(6, dtype=torch.float32).reshape(1, 6, 1) * 2 + 1      # 1,3,5,7,9,11
    plan = oracle.merge_plan(metric.bfloat16(), (1, 1, 6), (1, 1, 2), 2)
    assert list(plan["jstar"][0]) == [int(v) for v in vals["jstar"]]
    assert np.allclose(plan["u"][0][[1, 3, 5]], vals["u"], rtol=1e-12)
    assert list(plan["dst_of"][0]) == [int(v) for v in vals["dst_of"]]
    assert list(plan["pos"][0]) == [int(v) for v in vals["pos"]]
    y = oracle.merge_apply(x.bfloat16(), plan["dst_of"], plan["pos"], plan["Nm"])
    assert np.allclose(y[0, :, 0], vals["merged"], rtol=1e-13)
    back = oracle.bf16_to_f64(oracle.unmerge(oracle.round_to_bf16(y), plan["pos"]))
    assert np.allclose(back[0, :, 0], vals["unmerged"], rtol=1e-13)


# ---------------------------------------------------------------- matching inside nearby blocks
def _unit_descriptors(B, N, dm, seed):
    rng = np.random.default_rng(seed)
    m = rng.standard_normal((B, N, dm))
    return m / np.linalg.norm(m, axis=-1, keepdims=True)


def test_local_matching_with_a_window_over_the_whole_grid_is_the_global_matching():
    grid, part = (4, 6, 8), (2, 2, 2)
    mhat = _unit_descriptors(2, 4 * 6 * 8, 16, 1)
    sl_g, j_g, u_g, _ = oracle.merge_match(mhat, grid, part)
    sl_l, j_l, u_l, _ = oracle.merge_match_local(mhat, grid, part, (2, 3, 4))
    assert np.array_equal(sl_g, sl_l) and np.array_equal(j_g, j_l)
    assert np.allclose(u_g, u_l, rtol=0, atol=1e-14)


def test_local_matching_with_window_zero_picks_the_own_block():
    grid, part = (3, 5, 7), (2, 2, 3)
    mhat = _unit_descriptors(1, 3 * 5 * 7, 8, 2)
    sl, j, u, u2 = oracle.merge_match_local(mhat, grid, part, (0, 0, 0))
    i = sl[:, 1]
    t, rem = np.divmod(i, 5 * 7)
    y, x = np.divmod(rem, 7)
    own = ((t // 2 * 2) * 5 + y // 2 * 2) * 7 + x // 3 * 3
    assert np.array_equal(j, own)
    assert np.allclose(u, np.einsum("nd,nd->n", mhat[0, i], mhat[0, own]))
    assert np.all(np.isneginf(u2))


def test_local_matching_brute_force():
    grid, part, win = (3, 4, 6), (1, 2, 2), (1, 0, 1)
    T, Hh, W = grid
    mhat = _unit_descriptors(1, T * Hh * W, 8, 3)
    mhat[0, 7] = mhat[0, 1]          # a duplicated direction: exact tie between two destinations' scores
    is_dst = oracle.destination_mask(grid, part)
    sl, j, u, u2 = oracle.merge_match_local(mhat, grid, part, win)
    for (_, i), jj, uu, uu2 in zip(sl, j, u, u2):
        ti, yi, xi = i // (Hh * W), (i // W) % Hh, i % W
        cands = []
        for d in np.nonzero(is_dst)[0]:
            td, yd, xd = d // (Hh * W), (d // W) % Hh, d % W
            if (abs(td // 1 - ti // 1) <= win[0] and abs(yd // 2 - yi // 2) <= win[1]
                    and abs(xd // 2 - xi // 2) <= win[2]):
                cands.append((-float(mhat[0, i] @ mhat[0, d]), int(d)))
        cands.sort()
        assert jj == cands[0][1] and abs(uu + cands[0][0]) < 1e-14
        if len(cands) > 1:
            assert abs(uu2 + cands[1][0]) < 1e-14
