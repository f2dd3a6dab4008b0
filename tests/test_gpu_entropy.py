"""GPU-vs-oracle parity of the entropy-aware scheduler inputs (Sec. 3.4, Eq. 16-19).

Tolerances.  A weight is recomputed as exp(s - lse) from bf16 tensor-core logits and the fp32
log-sum-exp of the forward pass, whose own gate against the oracle is 2e-3 absolute: a weight can
be off by that relative amount, and so can a column sum of weights.  Gates: the marginal within
3e-3 relative to its largest entry (and summing to one within 3e-3), the entropy within 1e-3."""
import numpy as np
import pytest
import torch

import oracle
import usv_inputs as ui

DEV = "cuda:0"


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


CASES = [
    ("tiny", 1, 2, (4, 16, 16), 64, [4, 4]),
    ("ragged_d128", 2, 3, (10, 10, 10), 128, [3, 16, 7]),
    # several 128-key tiles per query tile of the tensor-core kernel and a partial last block
    # (8170 = 127 blocks of 64 + 42 tokens); per-head k from one block to a quarter of them
    ("mid_d128", 1, 4, (5, 38, 43), 128, [1, 13, 32, 7]),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_key_marginal_and_entropy(usv, case):
    name, B, H, grid, d, kph = case
    N = grid[0] * grid[1] * grid[2]
    wl = ui.workload("tiny") if name == "tiny" else ui.Workload(name, 100 + len(name), B, H, d, grid, (100,))
    q, k, v = ui.make_qkv(wl, device="cpu", layout="bhnd")
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    sel = usv.select_blocks(usv.block_scores(qd, kd, N, N), kph)
    _, lse = usv.sparse_attn_fwd(qd, kd, vd, sel, kph, N=N, return_lse=True)
    marg, ent = usv.attn_entropy(qd, kd, sel, kph, lse, N=N)
    torch.cuda.synchronize()
    m_ref = oracle.key_marginal(q, k, N, sel.cpu().numpy(), kph)
    h_ref = oracle.entropy(m_ref)
    m = marg.cpu().numpy().astype(np.float64)
    assert np.abs(m - m_ref).max() <= 3e-3 * m_ref.max()
    assert np.abs(m.sum(1) - 1.0).max() <= 3e-3
    assert np.abs(ent.cpu().numpy() - h_ref).max() <= 1e-3
    assert np.all((ent.cpu().numpy() >= 0) & (ent.cpu().numpy() <= 1 + 1e-6))
    print("%s: entropy %s (oracle %s)" % (name, ent.cpu().numpy(), h_ref))


def test_allocation_matches_oracle_and_rejects_bad_input():
    import paper_2512_05754_b200 as usv
    rng = np.random.default_rng(5)
    for L, gamma, rb, lo, hi in ((1, 1.0, 0.9, 0.0, 1.0), (12, 2.0, 0.8, 0.5, 0.95), (30, 3.5, 0.6, 0.1, 0.99)):
        h = rng.random(L).astype(np.float32)
        got = np.array(usv.allocate_sparsity(h, gamma, rb, lo, hi))
        ref = oracle.allocate(h.astype(np.float64), gamma, rb, lo, hi)
        assert np.abs(got - ref).max() <= 1e-6
    assert usv.allocate_sparsity([1.0, 1.0], 2.0, 0.7, 0.0, 1.0) == pytest.approx([0.7, 0.7])
    for bad in (([0.5, 1.5], 2.0), ([0.5], 0.5)):
        with pytest.raises(usv.USVError):
            usv.allocate_sparsity(bad[0], bad[1], 0.5, 0.0, 1.0)


@pytest.mark.gpu
def test_full_size_properties(usv):
    """Wan 480p shape, where the oracle's marginal is out of reach: what must hold at any size.
    Every row of attention weights sums to one, so the marginal sums to one; the entropy lies in
    [0,1]; keys of blocks that no query block selected carry exactly zero."""
    wl = ui.workload("wan1.3b_480p")
    q, k, v = ui.make_qkv(wl, device=DEV, layout="bhnd")
    kph, N = wl.k_per_head(), wl.N
    sel = usv.select_blocks(usv.block_scores(q, k, N, N), kph)
    _, lse = usv.sparse_attn_fwd(q, k, v, sel, kph, N=N, return_lse=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    usv.attn_entropy(q, k, sel, kph, lse, N=N)
    e0.record()
    marg, ent = usv.attn_entropy(q, k, sel, kph, lse, N=N)
    e1.record()
    torch.cuda.synchronize()
    assert abs(marg.sum().item() - 1.0) <= 3e-3
    assert 0.0 <= ent.item() <= 1.0
    used = torch.zeros(wl.NB, dtype=torch.bool, device=DEV)
    used[sel.flatten().long()] = True
    unused_keys = (~used).repeat_interleave(64)[:N]
    assert (marg[0][unused_keys] == 0).all()
    print("wan1.3b_480p: entropy %.6f, usv_attn_entropy %.3f ms" % (ent.item(), e0.elapsed_time(e1)))
