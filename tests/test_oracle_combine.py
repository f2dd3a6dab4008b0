"""Pins of the two-branch fusion of the oracle (oracle.attn_combine, select_blocks_long_range).

The Fig. 2 caption says only that the outputs of the local-cube branch and of the long-range
top-k branch are fused.  The reading taken (weights = softmax mass of each branch) is pinned by
what the mathematics fixes: it must reproduce ONE attention over the union of the two disjoint
key sets, which the oracle computes by an independent route (its masked dense attention)."""
import os

import numpy as np
import torch

import oracle
import usv_inputs as ui

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "combine_hand_example.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split("=")
            out[k.strip()] = np.array([float(x) for x in v.split()])
    return out


def test_hand_example():
    g = _golden()
    o, lse = oracle.attn_combine(g["o1"], g["lse1"][0], g["o2"], g["lse2"][0])
    assert np.allclose(o, g["o"], atol=1e-15) and abs(lse - g["lse"][0]) < 1e-15


def test_branch_without_keys_has_no_weight():
    o1, o2 = np.array([[3.0, -1.0]]), np.array([[7.0, 7.0]])
    o, lse = oracle.attn_combine(o1, np.array([0.3]), o2, np.array([-np.inf]))
    assert np.array_equal(o, o1) and lse[0] == 0.3
    o, lse = oracle.attn_combine(o1, np.array([-np.inf]), o2, np.array([-2.0]))
    assert np.array_equal(o, o2) and lse[0] == -2.0
    o, lse = oracle.attn_combine(o1, np.array([-np.inf]), o2, np.array([-np.inf]))
    assert np.array_equal(o, np.zeros((1, 2))) and lse[0] == -np.inf


def test_long_range_selection_excludes_the_own_block_and_matches_brute_force():
    rng = np.random.default_rng(3)
    s = rng.integers(-2, 3, size=(1, 2, 6, 6)).astype(np.float64)      # many exact ties
    kph = [2, 5]
    sel, _ = oracle.select_blocks_long_range(s, kph)
    import itertools
    for h, k in enumerate(kph):
        for i in range(6):
            others = [j for j in range(6) if j != i]
            best = max(itertools.combinations(others, k),
                       key=lambda c: (sum(s[0, h, i, j] for j in c), tuple(-j for j in c)))
            assert list(sel[0, h, i, :k]) == sorted(best) and i not in sel[0, h, i, :k]
    # only 5 other blocks exist: asking for more keeps all of them
    sel, _ = oracle.select_blocks_long_range(s[:, :1], [6])
    assert list(sel[0, 0, 2]) == [0, 1, 3, 4, 5, -1]


def test_fused_branches_equal_one_attention_over_the_union():
    """Local branch (own block) + long-range branch (k-1 other blocks), each through the oracle's
    sparse attention, fused: must equal the oracle's attention with the union selection, and the
    plain textbook softmax over exactly those keys."""
    wl = ui.Workload("combine", 91, 1, 2, 64, (3, 10, 13), (100,))          # 390 tokens, 7 blocks, ragged tail
    q, k, v = ui.make_qkv(wl)
    N, NB = wl.N, wl.NB
    kph = [3, 5]
    s = oracle.block_scores(oracle.block_pool(q, N), oracle.block_pool(k, N))
    sel_loc = np.arange(NB, dtype=np.int32).reshape(1, 1, NB, 1).repeat(2, 1)
    sel_lr, _ = oracle.select_blocks_long_range(s, [kk - 1 for kk in kph])
    sel_union, _ = oracle.select_blocks_local(s, kph)
    o1, l1 = oracle.sparse_attn(q, k, v, N, sel_loc, [1, 1])
    o2, l2 = oracle.sparse_attn(q, k, v, N, sel_lr, [kk - 1 for kk in kph])
    ou, lu = oracle.sparse_attn(q, k, v, N, sel_union, kph)
    o, lse = oracle.attn_combine(o1, l1, o2, l2)
    rows = np.arange(NB * 64).reshape(NB, 64) < N                           # valid query rows
    rows = np.tile(rows, (2, 1))
    assert np.abs(o - ou)[rows].max() < 1e-12 and np.abs(lse - lu)[rows].max() < 1e-12
    # swapping the two branches changes nothing; a wrong weighting (plain average) does
    o_sw, _ = oracle.attn_combine(o2, l2, o1, l1)
    assert np.abs(o_sw - o)[rows].max() < 1e-15
    assert np.abs(0.5 * (o1 + o2) - ou)[rows].max() > 1e-3
    # textbook check of one query row against a softmax over the union's keys, written out here
    h, I, r = 1, 2, 17
    keys = np.concatenate([np.arange(j * 64, min((j + 1) * 64, N)) for j in sel_union[0, h, I, :kph[h]]])
    qf, kf, vf = (t[0, h].double().numpy() for t in (q, k, v))
    logit = kf[keys] @ qf[I * 64 + r] / np.sqrt(wl.d)
    p = np.exp(logit - logit.max()); p /= p.sum()
    assert np.abs(p @ vf[keys] - o[h * NB + I, r]).max() < 1e-12
