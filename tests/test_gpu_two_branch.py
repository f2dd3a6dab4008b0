"""The two-branch form of Fig. 2 on the GPU: local-cube attention and long-range top-k attention
computed apart and fused (usv_exclude_own_block, usv_attn_combine), against the oracle's single
attention over the union of the two key sets.  Same gates as the attention parity tests."""
import numpy as np
import pytest
import torch

import oracle
import usv_inputs as ui
from parity_utils import attn_errors, check_selection

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MAX_ABS, REL_L2, REL_L2_BF16 = 2e-2, 1e-3, 2.5e-3


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


@pytest.mark.parametrize("d,B,H,grid,kph", [(128, 2, 3, (4, 12, 14), [4, 11, 2]), (64, 1, 2, (3, 9, 16), [3, 7])])
def test_two_branches_fused_equal_the_union_attention(usv, d, B, H, grid, kph):
    wl = ui.Workload("two_branch%d" % d, 140 + d, B, H, d, grid, (100,))
    q, k, v = ui.make_qkv(wl)
    N, NB = wl.N, wl.NB                                   # 672 / 432 tokens: partial last block
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    scores = usv.block_scores(qd, kd, N, N)
    # local branch: every query block attends its own block
    sel_loc = torch.arange(NB, dtype=torch.int32, device=DEV).view(1, 1, NB, 1).expand(B, H, NB, 1).contiguous()
    _, o1, l1 = usv.sparse_attn_fwd(qd, kd, vd, sel_loc, [1] * H, N=N, return_f32=True, return_lse=True)
    # long-range branch: the k - 1 best OTHER blocks
    s_lr = usv.exclude_own_block(scores.clone())
    assert torch.isinf(torch.diagonal(s_lr, dim1=2, dim2=3)).all() and (torch.diagonal(s_lr, dim1=2, dim2=3) < 0).all()
    k_lr = [kk - 1 for kk in kph]
    sel_lr = usv.select_blocks(s_lr, k_lr)
    _, o2, l2 = usv.sparse_attn_fwd(qd, kd, vd, sel_lr, k_lr, N=N, return_f32=True, return_lse=True)
    o, o32, lse = usv.attn_combine(o1, l1, o2, l2, return_f32=True, return_lse=True)
    torch.cuda.synchronize()
    assert usv.workspace_status() == 0
    # the long-range selection against the oracle's (bit-exact outside the near-tie band)
    s_ref = oracle.block_scores(oracle.block_pool(q, N), oracle.block_pool(k, N))
    ref_lr, gap = oracle.select_blocks_long_range(s_ref, k_lr)
    got_lr = sel_lr.cpu().numpy()
    same = (got_lr == ref_lr).all(-1)
    assert np.all(same | (gap < 1e-3))
    for h in range(H):
        own = np.arange(NB)[None, :, None]
        assert not (got_lr[:, h, :, :k_lr[h]] == own).any(), "own block selected by the long-range branch"
    # fused output against ONE oracle attention over own block + the GPU's long-range blocks
    union = np.full((B, H, NB, max(kph)), -1, dtype=np.int32)
    for b in range(B):
        for h in range(H):
            for i in range(NB):
                union[b, h, i, :kph[h]] = sorted(list(got_lr[b, h, i, :k_lr[h]]) + [i])
    o_ref, lse_ref = oracle.sparse_attn(q, k, v, N, union, kph)
    o_ref = o_ref.reshape(B, H, NB * 64, d)[:, :, :N]
    lse_ref = lse_ref.reshape(B, H, NB * 64)[:, :, :N]
    mx, rl2 = attn_errors(o32.cpu().numpy(), o_ref)
    _, rl2b = attn_errors(o.float().cpu().numpy(), o_ref)
    print("two-branch d=%d: max-abs %.3g rel-L2 %.3g (bf16 %.3g)" % (d, mx, rl2, rl2b))
    assert mx <= MAX_ABS and rl2 <= REL_L2 and rl2b <= REL_L2_BF16
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 2e-3
    assert torch.equal(o.cpu(), o32.to(torch.bfloat16).cpu())
    # the combine step alone, element by element against the oracle's formula on the same inputs
    oc, lc = oracle.attn_combine(o1.cpu().numpy(), l1.cpu().numpy(), o2.cpu().numpy(), l2.cpu().numpy())
    assert np.abs(o32.cpu().numpy() - oc).max() <= 2e-6 * max(1.0, np.abs(oc).max())
    assert np.abs(lse.cpu().numpy() - lc).max() <= 2e-6 * max(1.0, np.abs(lc).max())
    # bf16 branch outputs as inputs (what a bf16 pipeline hands over)
    ob = usv.attn_combine(o1.to(torch.bfloat16), l1, o2.to(torch.bfloat16), l2)
    _, rl2c = attn_errors(ob.float().cpu().numpy(), o_ref)
    assert rl2c <= 2 * REL_L2_BF16


def test_combine_ignores_an_empty_branch(usv):
    B, H, N, d = 1, 2, 70, 128
    g = torch.Generator().manual_seed(4)
    o1 = torch.randn(B, H, N, d, generator=g).to(DEV)
    o2 = torch.full((B, H, N, d), float("nan"), device=DEV)
    l1 = torch.randn(B, H, N, generator=g).to(DEV)
    l2 = torch.full((B, H, N), float("-inf"), device=DEV)
    o, o32, lse = usv.attn_combine(o1, l1, o2, l2, return_f32=True, return_lse=True)
    assert torch.equal(o32, o1) and torch.equal(lse, l1)
    o, o32, lse = usv.attn_combine(o2, l2, o2, l2, return_f32=True, return_lse=True)
    assert torch.equal(o32, torch.zeros_like(o32)) and torch.isinf(lse).all()
