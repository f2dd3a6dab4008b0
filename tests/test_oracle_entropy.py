"""Pins of the oracle's entropy-aware scheduler functions (Sec. 3.4, Eq. 16-19): hand-worked
values, closed forms, and the dense special case against a textbook softmax."""
import os

import numpy as np
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "entropy_hand_example.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        if line.startswith("#") or "=" not in line:
            continue
        k, v = line.split("=")
        out[k.strip()] = np.array([float(x) for x in v.split()])
    return out


def _bf16(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)


def test_entropy_hand_example_and_extremes():
    g = _gold()
    assert abs(oracle.entropy(np.array([[0.5, 0.25, 0.25]]))[0] - g["h_example"][0]) < 1e-15
    n = 37
    assert abs(oracle.entropy(np.full((1, n), 1.0 / n))[0] - 1.0) < 1e-14        # uniform marginal: h = 1
    one_hot = np.zeros((1, n)); one_hot[0, 5] = 1.0
    assert oracle.entropy(one_hot)[0] == 0.0                                      # all mass on one key: h = 0
    # permuting the keys does not change the entropy
    rng = np.random.default_rng(0)
    a = rng.random((1, n)); a /= a.sum()
    assert abs(oracle.entropy(a)[0] - oracle.entropy(a[:, rng.permutation(n)])[0]) < 1e-14


def test_allocation_hand_examples_and_budget():
    g = _gold()
    h = np.array([0.0, 0.5])
    assert np.allclose(oracle.allocate(h, 1.0, 0.6, 0.0, 10.0), g["rho_gamma1"], atol=1e-15)
    assert np.allclose(oracle.allocate(h, 2.0, 0.6, 0.0, 10.0), g["rho_gamma2"], atol=1e-15)
    assert np.allclose(oracle.allocate(h, 2.0, 0.6, 0.3, 0.9), g["rho_gamma2_clipped"], atol=1e-15)
    # equal entropies: every layer gets the base ratio; without clipping the mean is the budget
    assert np.allclose(oracle.allocate(np.full(7, 0.3), 3.0, 0.8, 0.0, 1.0), 0.8)
    rng = np.random.default_rng(1)
    hh = rng.random(12) * 0.9
    assert abs(oracle.allocate(hh, 2.0, 0.5, 0.0, 100.0).mean() - 0.5) < 1e-14
    # lower entropy => at least as much sparsity
    r = oracle.allocate(np.sort(hh), 1.5, 0.5, 0.0, 100.0)
    assert np.all(np.diff(r) <= 1e-15)


def test_key_marginal_closed_forms():
    B, H, N, d = 1, 2, 100, 64            # two blocks, the second partial (36 valid keys)
    sel = np.array([[[[0, 1], [0, 1]]] * H], dtype=np.int32).reshape(B, H, 2, 2)
    k = _bf16(np.random.default_rng(2).standard_normal((B, H, N, d)))
    # zero queries: every row is uniform over its N allowed keys -> uniform marginal, h = 1
    m = oracle.key_marginal(_bf16(np.zeros((B, H, N, d))), k, N, sel, [2, 2])
    assert np.allclose(m, 1.0 / N, atol=1e-15) and abs(oracle.entropy(m)[0] - 1.0) < 1e-13
    # each query block only sees key block 1: keys 0..63 get no mass, the marginal still sums to one
    sel1 = np.array([1, -1] * (H * 2), dtype=np.int32).reshape(B, H, 2, 2)
    m1 = oracle.key_marginal(_bf16(np.zeros((B, H, N, d))), k, N, sel1, [1, 1])
    assert np.all(m1[0, :64] == 0.0) and np.allclose(m1[0, 64:], 1.0 / 36, atol=1e-15)
    # one key dominates every row: the marginal concentrates there, h -> 0
    q = np.zeros((B, H, N, d)); q[..., 0] = 16.0
    kk = np.zeros((B, H, N, d)); kk[:, :, 7, 0] = 16.0
    m2 = oracle.key_marginal(_bf16(q), _bf16(kk), N, sel, [2, 2], scale=1.0)
    assert m2[0, 7] > 1.0 - 1e-12 and oracle.entropy(m2)[0] < 1e-12


def test_key_marginal_dense_case_matches_textbook_softmax():
    B, H, N, d = 2, 3, 128, 64
    rng = np.random.default_rng(3)
    q = _bf16(rng.standard_normal((B, H, N, d)))
    k = _bf16(rng.standard_normal((B, H, N, d)))
    sel = np.tile(np.arange(2, dtype=np.int32), (B, H, 2, 1))
    m = oracle.key_marginal(q, k, N, sel, [2] * H)
    a = torch.softmax(q.double() @ k.double().transpose(-1, -2) / d ** 0.5, -1)   # [B,H,N,N]
    ref = a.mean(dim=(1, 2)).numpy()
    assert np.abs(m - ref).max() < 1e-15
    assert np.allclose(m.sum(1), 1.0, atol=1e-13)
    # a sparse mask: masked columns carry exactly zero weight in rows that do not select them
    sel_s = np.array([[0, -1], [1, -1]], dtype=np.int32)[None, None].repeat(B, 0).repeat(H, 1)
    ms = oracle.key_marginal(q, k, N, sel_s, [1] * H)
    a0 = torch.softmax(q[:, :, :64].double() @ k[:, :, :64].double().transpose(-1, -2) / d ** 0.5, -1)
    assert np.abs(ms[:, :64] - a0.sum(dim=(1, 2)).numpy() / (H * N)).max() < 1e-15
