"""Attention with the unmerge folded into its epilogue (usv_sparse_attn_fwd_unmerge) against
oracle.unmerge(oracle attention), and bit for bit against the two-call path it replaces."""
import numpy as np
import pytest
import torch

import oracle
import usv_inputs as ui
from parity_utils import attn_errors, bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MAX_ABS, REL_L2_BF16 = 2e-2, 2.5e-3


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


def test_unmerge_map_is_the_inverse_of_pos(usv):
    g = torch.Generator().manual_seed(2)
    B, N, Nm = 3, 1000, 377
    pos = torch.randint(0, Nm, (B, N), generator=g, dtype=torch.int32)
    pos[:, :Nm] = torch.arange(Nm, dtype=torch.int32)            # every merged row is read at least once
    off, idx = usv.unmerge_map(pos.to(DEV), Nm)
    off, idx = off.cpu().numpy(), idx.cpu().numpy()
    p = pos.numpy()
    for b in range(B):
        assert off[b, 0] == 0 and off[b, Nm] == N and (np.diff(off[b]) >= 1).all()
        assert sorted(idx[b]) == list(range(N))
        for m in (0, 1, 17, Nm - 1):
            assert sorted(idx[b, off[b, m]:off[b, m + 1]]) == list(np.nonzero(p[b] == m)[0])


@pytest.mark.parametrize("B,H,grid,part,r,kph", [(2, 3, (4, 10, 12), (1, 1, 2), 150, [3, 6, 5]),
                                                 (1, 2, (3, 9, 14), (1, 2, 2), 201, [2, 3])])
def test_fused_unmerge_matches_oracle_and_the_two_call_path(usv, B, H, grid, part, r, kph):
    d = 128
    wl = ui.Workload("fused_unmerge", 170 + H, B, H, d, grid, (100,))
    N_full = wl.N
    z = ui.make_hidden(wl, DEV)                                               # [B,N,C]
    metric = z.reshape(B, N_full, H, d).contiguous()
    zm, plan = usv.token_merge(z, metric, grid, part, r)
    N = N_full - r
    g = torch.Generator().manual_seed(5)
    w = (torch.randn(wl.C, 3 * wl.C, generator=g) / wl.C ** 0.5).to(torch.bfloat16).to(DEV)
    qkv = (zm @ w).reshape(B, N, 3, H, d)
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    sel = usv.select_blocks(usv.block_scores(q, k, N, N), kph)
    # two calls: attention on the merged sequence, then the gather
    o = usv.sparse_attn_fwd(q, k, v, sel, kph, N=N)
    y_ref_gpu = usv.token_unmerge(o.permute(0, 2, 1, 3).reshape(B, N, wl.C), plan.pos)
    # one call
    umap = usv.unmerge_map(plan.pos, N)
    y, o32 = usv.sparse_attn_fwd_unmerge(q, k, v, sel, kph, umap, N_full, N=N, return_f32=True)
    torch.cuda.synchronize()
    assert usv.workspace_status() == 0
    assert torch.equal(y.view(torch.int16), y_ref_gpu.view(torch.int16)), "fused unmerge differs from attention + unmerge"
    # against the oracle: attention on the merged sequence (GPU's selection), rounded to bf16, unmerged
    o_ref, _ = oracle.sparse_attn(q.cpu(), k.cpu(), v.cpu(), N, sel.cpu().numpy(), kph)
    NB = (N + 63) // 64
    o_ref = o_ref.reshape(B, H, NB * 64, d)[:, :, :N]
    om_bits = oracle.round_to_bf16(np.ascontiguousarray(o_ref.transpose(0, 2, 1, 3).reshape(B, N, wl.C)))
    y_ref = oracle.bf16_to_f64(oracle.unmerge(om_bits, plan.pos.cpu().numpy()))       # Eq. 15 on the oracle's output
    mx, rl2 = attn_errors(y.float().cpu().numpy(), y_ref)
    print("fused unmerge: max-abs %.3g rel-L2 (bf16) %.3g" % (mx, rl2))
    assert mx <= MAX_ABS and rl2 <= REL_L2_BF16
    assert torch.equal(o.permute(0, 2, 1, 3).reshape(B, N, wl.C).cpu(),
                       o32.to(torch.bfloat16).permute(0, 2, 1, 3).reshape(B, N, wl.C).cpu())
