"""Pins of the CPU oracle's coarse-selection and attention functions against things other than
itself: library dense softmax attention, closed forms, brute-force enumeration, invariants and
the hand-derived values stored under tests/golden/."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
import usv_inputs as ui

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


def _f64(x):
    return x.to(torch.float64).numpy()


def _numpy_dense_attention(q, k, v, scale):
    """Textbook softmax(QK^T * scale) V with numpy library routines, fp64."""
    s = np.einsum("bhid,bhjd->bhij", q, k) * scale
    s = s - s.max(-1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(-1, keepdims=True)
    return np.einsum("bhij,bhjd->bhid", p, v)


# ------------------------------------------------------------------ bf16 helpers

def test_bf16_roundtrip_and_rne():
    # every finite bf16 pattern survives bits -> double -> bits
    bits = np.arange(0, 0x10000, dtype=np.uint32).astype(np.uint16)
    finite = (bits & 0x7f80) != 0x7f80
    back = oracle.round_to_bf16(oracle.bf16_to_f64(bits[finite]))
    assert np.array_equal(back, bits[finite])
    # ties go to the even significand; values just off a tie go to the nearer neighbour
    x = np.array([1 + 2.0**-8, 1 + 3 * 2.0**-8, 1 + 2.0**-8 + 2.0**-30, 1 + 3 * 2.0**-8 - 2.0**-30])
    assert [hex(b) for b in oracle.round_to_bf16(x)] == ["0x3f80", "0x3f82", "0x3f81", "0x3f81"]
    # agrees with torch's float32 -> bf16 conversion on float32 inputs (one rounding each)
    g = torch.Generator().manual_seed(3)
    f = torch.randn(20000, generator=g) * torch.exp(torch.randn(20000, generator=g) * 8)
    ref = f.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.round_to_bf16(f.to(torch.float64).numpy()), ref)


# ------------------------------------------------------------------ pooling and scores

def test_block_pool_constant_blocks_and_partial_tail():
    B, H, N, d = 1, 2, 64 * 3 + 2, 8
    x = torch.zeros(B, H, N, d)
    for I in range(4):
        x[:, :, I * 64:(I + 1) * 64, :] = float(I + 1)
    x[0, 1, 192, :] = 3.0      # the two valid tokens of the last block of head 1: 3 and 5
    x[0, 1, 193, :] = 5.0
    xb = x.to(torch.bfloat16)
    p = oracle.block_pool(xb, N)
    assert p.shape == (B, H, 4, d)
    assert np.allclose(p[0, 0, :, 0], [1, 2, 3, 4], atol=0)
    assert p[0, 1, 3, 0] == 4.0          # (3 + 5) / 2: divides by the valid count, not by 64


def test_block_pool_matches_numpy_mean_with_strides():
    B, H, N, d = 2, 3, 200, 16
    mem = _rand_bf16((B, N, H, d), 5)          # token-major memory, permuted view
    view = mem.permute(0, 2, 1, 3)
    p = oracle.block_pool(view, N)
    ref = _f64(view)
    for I in range(4):
        lo, hi = I * 64, min(N, I * 64 + 64)
        assert np.allclose(p[:, :, I], ref[:, :, lo:hi].mean(2), rtol=1e-13, atol=1e-15)


def test_block_scores_is_scaled_gram_matrix():
    rng = np.random.default_rng(0)
    qb = rng.standard_normal((2, 2, 5, 16))
    kb = rng.standard_normal((2, 2, 7, 16))
    s = oracle.block_scores(qb, kb)
    ref = np.einsum("bhid,bhjd->bhij", qb, kb) / 4.0        # sqrt(16) = 4
    assert s.shape == (2, 2, 5, 7)
    assert np.allclose(s, ref, rtol=1e-13, atol=1e-15)
    # not symmetric in its operands: transposing the roles must change the answer
    assert not np.allclose(s[..., :5, :5], np.swapaxes(s[..., :5, :5], -1, -2))


# ------------------------------------------------------------------ top-k selection

@pytest.mark.parametrize("NB,k", [(6, 1), (6, 3), (8, 4), (7, 7)])
def test_select_blocks_brute_force(NB, k):
    rng = np.random.default_rng(NB * 10 + k)
    s = rng.standard_normal((1, 2, 5, NB))
    s[0, 0, 0, :] = 0.25                       # a fully tied row
    s[0, 1, 2, 1] = s[0, 1, 2, 4]              # a tie that may straddle the cut
    sel, gap = oracle.select_blocks(s, [k, k])
    for h in range(2):
        for I in range(5):
            row = s[0, h, I]
            best, best_sum = None, -np.inf
            for sub in itertools.combinations(range(NB), k):   # lexicographic order
                t = row[list(sub)].sum()
                if t > best_sum + 1e-15:
                    best, best_sum = sub, t
            assert tuple(sel[0, h, I]) == best, (h, I)
            srt = np.sort(row)[::-1]
            if k < NB:
                g = (srt[k - 1] - srt[k]) / max(abs(srt[k - 1]), abs(srt[k]), 1e-30)
                assert np.isclose(gap[0, h, I], g)
            else:
                assert np.isinf(gap[0, h, I])


def test_select_blocks_special_cases():
    rng = np.random.default_rng(1)
    s = rng.standard_normal((1, 3, 4, 10))
    # k = NB keeps everything, in order
    sel, _ = oracle.select_blocks(s, [10, 10, 10])
    assert np.array_equal(sel, np.broadcast_to(np.arange(10), sel.shape))
    # constant scores: lowest indices win
    sel, gap = oracle.select_blocks(np.ones((1, 3, 4, 10)), [3, 3, 3])
    assert np.array_equal(sel, np.broadcast_to(np.arange(3), sel.shape))
    assert np.all(gap == 0)
    # adding a per-row constant does not change the selection; per-head k with a -1 tail
    sel_a, _ = oracle.select_blocks(s, [2, 5, 1], kmax=6)
    sel_b, _ = oracle.select_blocks(s + rng.standard_normal((1, 3, 4, 1)), [2, 5, 1], kmax=6)
    assert np.array_equal(sel_a, sel_b)
    assert np.all(sel_a[0, 0, :, 2:] == -1) and np.all(sel_a[0, 1, :, 5:] == -1)
    assert np.all(sel_a[0, 2, :, 0] == s[0, 2].argmax(-1))
    assert np.all(np.diff(sel_a[0, 1, :, :5], axis=-1) > 0)      # ascending block index


# ------------------------------------------------------------------ attention values

def test_keep_all_equals_library_dense_attention():
    B, H, N, d = 1, 2, 256, 32
    q, k, v = (_rand_bf16((B, H, N, d), s) for s in (10, 11, 12))
    NB = N // 64
    sel = np.broadcast_to(np.arange(NB, dtype=np.int32), (B, H, NB, NB)).copy()
    ref = _numpy_dense_attention(_f64(q), _f64(k), _f64(v), 1 / np.sqrt(d))
    o_dense, rowsum = oracle.dense_masked_attn(q, k, v, N, sel, [NB] * H)
    o_sparse, lse = oracle.sparse_attn(q, k, v, N, sel, [NB] * H)
    assert np.allclose(o_dense, ref, rtol=1e-12, atol=1e-14)
    assert np.allclose(o_sparse.reshape(B, H, N, d), ref, rtol=1e-12, atol=1e-14)
    assert np.allclose(rowsum, 1.0, atol=1e-14)
    s = np.einsum("bhid,bhjd->bhij", _f64(q), _f64(k)) / np.sqrt(d)
    ref_lse = np.log(np.exp(s).sum(-1))
    assert np.allclose(lse.reshape(B, H, N), ref_lse, rtol=1e-12)


def test_restricted_evaluation_equals_literal_mask_on_tiny_workload():
    wl = ui.workload("tiny")
    q, k, v = ui.make_qkv(wl)
    N, NB, kph = wl.N, wl.NB, wl.k_per_head()
    scores = oracle.block_scores(oracle.block_pool(q, N), oracle.block_pool(k, N))
    sel, _ = oracle.select_blocks(scores, kph)
    o_dense, rowsum = oracle.dense_masked_attn(q, k, v, N, sel, kph)
    o_sparse, _ = oracle.sparse_attn(q, k, v, N, sel, kph)
    assert np.allclose(rowsum, 1.0, atol=1e-13)
    assert np.allclose(o_sparse.reshape(o_dense.shape), o_dense, rtol=1e-11, atol=1e-13)
    # and the literal mask agrees with a numpy evaluation of the masked formula
    mask = np.zeros((wl.B, wl.H, N, N), dtype=bool)
    for h in range(wl.H):
        for I in range(NB):
            for J in sel[0, h, I]:
                mask[0, h, I * 64:(I + 1) * 64, J * 64:(J + 1) * 64] = True
    s = np.einsum("bhid,bhjd->bhij", _f64(q), _f64(k)) / np.sqrt(wl.d)
    s = np.where(mask, s, -np.inf)
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    assert np.allclose(o_dense, np.einsum("bhij,bhjd->bhid", p, _f64(v)), rtol=1e-11, atol=1e-13)


def test_masked_blocks_contribute_nothing_and_block_permutation_invariance():
    B, H, N, d = 1, 1, 320, 16
    q, k, v = (_rand_bf16((B, H, N, d), s) for s in (20, 21, 22))
    NB = 5
    sel = np.array([[0, 3], [1, 2], [0, 4], [2, 3], [1, 4]], dtype=np.int32).reshape(1, 1, NB, 2)
    o, _ = oracle.sparse_attn(q, k, v, N, sel, [2])
    # poison keys/values of a block nobody selected for query block 0 (blocks 1,2,4)
    k2, v2 = k.clone(), v.clone()
    k2[0, 0, 64:192] = 7.0
    v2[0, 0, 64:192] = -9.0
    o2, _ = oracle.sparse_attn(q, k2, v2, N, sel, [2])
    assert np.array_equal(o[0], o2[0])
    assert not np.array_equal(o[1], o2[1])
    # permuting key blocks (with V) and relabelling the selection leaves O unchanged
    perm = np.array([3, 0, 4, 1, 2])            # new block b holds old block perm[b]
    inv = np.argsort(perm)
    idx = (perm[:, None] * 64 + np.arange(64)[None, :]).reshape(-1)
    kp, vp = k[:, :, idx], v[:, :, idx]
    selp = np.sort(inv[sel], axis=-1).astype(np.int32)
    op, _ = oracle.sparse_attn(q, kp, vp, N, selp, [2])
    assert np.allclose(op, o, rtol=1e-12, atol=1e-14)


def test_pad_keys_are_masked_and_pad_rows_zero():
    B, H, N, d = 1, 1, 100, 16                  # second block has 36 valid tokens
    q, k, v = (_rand_bf16((B, H, 128, d), s) for s in (30, 31, 32))
    k[0, 0, N:] = 50.0                          # garbage in the pad rows must not matter
    v[0, 0, N:] = 50.0
    sel = np.array([[0, 1], [0, 1]], dtype=np.int32).reshape(1, 1, 2, 2)
    o, lse = oracle.sparse_attn(q, k, v, N, sel, [2])
    ref = _numpy_dense_attention(_f64(q)[:, :, :N], _f64(k)[:, :, :N], _f64(v)[:, :, :N], 0.25)
    assert np.allclose(o.reshape(128, d)[:N], ref[0, 0], rtol=1e-12, atol=1e-14)
    assert np.all(o.reshape(128, d)[N:] == 0) and np.all(lse.reshape(128)[N:] == 0)


def test_hand_worked_attention_example():
    """Two keys per query with logits chosen so that the softmax weights are exact fractions;
    expected outputs derived by hand in tests/golden/attention_hand_example.txt."""
    path = os.path.join(GOLDEN, "attention_hand_example.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    expected = np.array([[float(x) for x in r] for r in rows])
    N, d = 128, 2
    q = torch.zeros(1, 1, N, d)
    k = torch.zeros(1, 1, N, d)
    v = torch.zeros(1, 1, N, d)
    q[0, 0, :, 0] = 1.0
    # block 0 keys all have logit 0 except key 0 (logit ln 3 -> bf16 exact value used below)
    k[0, 0, 0, 0] = 2.0                      # scaled logit = 2 * scale
    v[0, 0, 0] = torch.tensor([1.0, 0.0])
    v[0, 0, 1:64] = torch.tensor([0.0, 1.0])
    v[0, 0, 64:] = torch.tensor([4.0, 4.0])
    sel = np.array([[0], [1]], dtype=np.int32).reshape(1, 1, 2, 1)
    scale = np.log(63.0) / 2.0               # key 0 weighs exp(ln 63) = 63 against 63 ones
    o, lse = oracle.sparse_attn(q.bfloat16(), k.bfloat16(), v.bfloat16(), N, sel, [1], scale=scale)
    assert np.allclose(o[0, 0], expected[0], rtol=1e-13)        # query block 0 -> [1/2, 1/2]
    assert np.allclose(o[1, 5], expected[1], rtol=1e-13)        # query block 1 -> [4, 4]
    assert np.isclose(lse[0, 0], expected[2, 0], rtol=1e-13)    # ln(126)
    assert np.isclose(lse[1, 0], expected[2, 1], rtol=1e-13)    # ln(64)
