"""GPU-vs-oracle parity of the cube token order and of the selection with the own block forced in
(overview figure of the paper: local 3D cubes, local cube attention beside the top-k selection).

Index work: bit-exact.  The forced selection is compared on the oracle's fp64 evaluation of the
GPU's own fp32 scores, so a row may differ only inside the near-tie band of the other tests."""
import numpy as np
import pytest
import torch

import oracle
import usv_inputs as ui

DEV = "cuda:0"
BAND = 1e-3


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


GRIDS = [
    ((1, 2, 3), (1, 2, 2)),          # the hand-worked grid of the oracle's pins
    ((8, 12, 16), (4, 4, 4)),        # whole cubes only
    ((5, 6, 7), (4, 4, 4)),          # every edge cuts a cube
    ((21, 30, 52), (4, 4, 4)),       # the Wan 480p latent grid: 32 760 tokens, several hundred launch blocks
    ((3, 9, 10), (2, 4, 3)),
    ((2, 3, 4), (7, 7, 7)),          # one cube larger than the grid: raster order
]


@pytest.mark.gpu
@pytest.mark.parametrize("grid,cube", GRIDS, ids=["%dx%dx%d_%dx%dx%d" % (g + c) for g, c in GRIDS])
def test_cube_order_matches_the_oracle(usv, grid, cube):
    perm, inv = usv.cube_order(grid, cube, device=DEV)
    torch.cuda.synchronize()
    perm_ref, inv_ref = oracle.cube_order(grid, cube)
    assert np.array_equal(perm.cpu().numpy(), perm_ref)
    assert np.array_equal(inv.cpu().numpy(), inv_ref)
    perm_only, none = usv.cube_order(grid, cube, device=DEV, want_inverse=False)
    assert none is None and torch.equal(perm_only, perm)


@pytest.mark.gpu
def test_tokens_go_into_cube_order_and_back(usv):
    grid = (5, 6, 7)
    n = grid[0] * grid[1] * grid[2]
    g = torch.Generator().manual_seed(3)
    x = torch.randn((2, n, 64), generator=g).to(torch.bfloat16).to(DEV)
    perm, inv = usv.cube_order(grid, (4, 4, 4), device=DEV)
    y = usv.permute_tokens(x, perm)
    back = usv.permute_tokens(y, inv)
    torch.cuda.synchronize()
    perm_ref, _ = oracle.cube_order(grid, (4, 4, 4))
    assert torch.equal(y.cpu(), x.cpu()[:, torch.from_numpy(perm_ref.astype(np.int64)), :])
    assert torch.equal(back, x)


def _check_local(sel_gpu, scores64, kph):
    sel_ref, gap = oracle.select_blocks_local(scores64, kph)
    B, H, NBq, NBk = scores64.shape
    differing = 0
    for h in range(H):
        k = int(kph[h])
        g, r = sel_gpu[:, h, :, :k], sel_ref[:, h, :, :k]
        assert np.all(sel_gpu[:, h, :, k:] == -1)
        if k > 1:
            assert np.all(np.diff(g, axis=-1) > 0)
        for b in range(B):
            for i in range(NBq):
                if i < NBk:
                    assert i in g[b, i], "the own block must be kept"
                if np.array_equal(g[b, i], r[b, i]):
                    continue
                differing += 1
                assert gap[b, h, i] < BAND, "selection differs outside the near-tie band"
    return differing


@pytest.mark.gpu
@pytest.mark.parametrize("case", [("tiny", (4, 16, 16), 64, 2, [4, 1]), ("mid_d128", (6, 20, 32), 128, 3, [7, 60, 1])],
                         ids=["tiny", "mid_d128"])
def test_forced_own_block_selection(usv, case):
    name, grid, d, H, kph = case
    wl = ui.Workload(name, 300 + len(name), 1, H, d, grid, (100,))
    q, k, _ = ui.make_qkv(wl, device=DEV, layout="bhnd")
    N = wl.N
    s = usv.block_scores(q, k, N, N)
    s64 = s.double().cpu().numpy().copy()          # the scores before the diagonal is raised
    usv.force_own_block(s)
    sel = usv.select_blocks(s, kph)
    torch.cuda.synchronize()
    NB = s.shape[2]
    diag = s.cpu().numpy()[0, :, np.arange(NB), np.arange(NB)]
    assert np.all(np.isposinf(diag))
    off = s.cpu().numpy().copy()
    off[0, :, np.arange(NB), np.arange(NB)] = s64[0, :, np.arange(NB), np.arange(NB)].astype(np.float32)
    assert np.array_equal(off, s64.astype(np.float32)), "only the diagonal may change"
    _check_local(sel.cpu().numpy(), s64, kph)


@pytest.mark.gpu
def test_cube_ordered_attention_keeps_the_own_cube(usv):
    """The whole local + long-range step on cube-ordered tokens: permute, score, force, select,
    attend; every query block attends its own cube, and the result matches the oracle's
    attention for the selection the GPU made."""
    grid, d, H, kph = (8, 8, 8), 64, 2, [3, 3]
    wl = ui.Workload("cubes_e2e", 321, 1, H, d, grid, (100,))
    q, k, v = ui.make_qkv(wl, device=DEV, layout="bnhd")     # token-major: [B,N,H*d] rows
    N = wl.N
    perm, inv = usv.cube_order(grid, (4, 4, 4), device=DEV)

    def to_cubes(t):                                          # t: [B,H,N,d] view of a [B,N,H,d] tensor
        flat = t.permute(0, 2, 1, 3).reshape(1, N, H * d).contiguous()
        return usv.permute_tokens(flat, perm).view(1, N, H, d).permute(0, 2, 1, 3)
    qc, kc, vc = to_cubes(q), to_cubes(k), to_cubes(v)
    s = usv.block_scores(qc, kc, N, N)
    usv.force_own_block(s)
    sel = usv.select_blocks(s, kph)
    o, o32 = usv.sparse_attn_fwd(qc, kc, vc, sel, kph, N=N, return_f32=True)
    torch.cuda.synchronize()
    sel_np = sel.cpu().numpy()
    NB = N // 64
    for i in range(NB):
        assert i in sel_np[0, 0, i] and i in sel_np[0, 1, i]
    ref, _ = oracle.sparse_attn(qc.contiguous().cpu(), kc.contiguous().cpu(), vc.contiguous().cpu(), N, sel_np, kph)
    got = o32.cpu().numpy().astype(np.float64).reshape(1 * H * NB, 64, d)     # (b, h, I) order, as the oracle's
    err = np.abs(got - ref)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert err.max() <= 2e-2 and rel <= 1e-3
