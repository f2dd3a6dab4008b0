"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

Integer outputs (block selections, merge plans) are checked in full or on seeded samples;
attention values on seeded samples of query blocks that the oracle computes one by one."""
import numpy as np
import pytest
import torch

import oracle
import usv_inputs as ui
from parity_utils import (attn_errors, bf16_ulp_distance, bits, check_merge_plan, check_selection,
                          gather_qblocks)

pytestmark = pytest.mark.gpu
MAX_ABS, REL_L2, REL_L2_BF16 = 2e-2, 1e-3, 2.5e-3
DEV = "cuda:0"


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


def _sample_qblocks(B, H, NB, n, seed, always=()):
    rng = np.random.default_rng(seed)
    allqb = oracle.all_query_blocks(B, H, NB)
    pick = rng.choice(allqb.shape[0], size=min(n, allqb.shape[0]), replace=False)
    qb = [tuple(r) for r in allqb[np.sort(pick)]]
    for extra in always:
        if extra not in qb:
            qb.append(extra)
    return np.array(qb, dtype=np.int32)


def _attention_parity(usv, q, k, v, N, kph, n_sample, seed, check_sel=True):
    """q,k,v: CUDA bf16 [B,H,N,d] views.  Runs A1-A4 on the GPU and compares with the oracle."""
    B, H, _, d = q.shape
    NB = (N + 63) // 64
    scores = usv.block_scores(q, k, N, N)
    sel = usv.select_blocks(scores, kph)
    o, o32 = usv.sparse_attn_fwd(q, k, v, sel, kph, N=N, return_f32=True)
    torch.cuda.synchronize()
    assert usv.workspace_status() == 0
    print("query blocks recomputed by the exact kernel: %d" % usv.sparse_attn_fallbacks())
    qc, kc, vc = (t.cpu() for t in (q, k, v))
    sel_np = sel.cpu().numpy()
    if check_sel:
        s_ref = oracle.block_scores(oracle.block_pool(qc, N), oracle.block_pool(kc, N))
        assert np.abs(scores.cpu().numpy() - s_ref).max() <= 2e-6 * max(1.0, np.abs(s_ref).max())
        rows, amb, diff = check_selection(sel_np, s_ref, kph)
        print("selection: %d rows, %d inside the near-tie band, %d differ" % (rows, amb, diff))
    # sample query blocks; always include the last (partial) block of the first and last head
    qb = _sample_qblocks(B, H, NB, n_sample, seed, always=[(0, 0, NB - 1), (B - 1, H - 1, NB - 1), (0, 0, 0)])
    o_ref, _ = oracle.sparse_attn(qc, kc, vc, N, sel_np, kph, qb_list=qb)
    got32 = gather_qblocks(o32, qb, N)
    got16 = gather_qblocks(o, qb, N)
    mx, rl2 = attn_errors(got32, o_ref)
    _, rl2b = attn_errors(got16, o_ref)
    print("attention on %d sampled query blocks: max-abs %.3g rel-L2 %.3g (bf16 %.3g)" % (len(qb), mx, rl2, rl2b))
    assert mx <= MAX_ABS and rl2 <= REL_L2 and rl2b <= REL_L2_BF16
    assert torch.equal(o, o32.to(torch.bfloat16)), "bf16 output != RNE(fp32 output)"
    return o


def test_wan_480p(usv):
    wl = ui.workload("wan1.3b_480p")
    q, k, v = ui.make_qkv(wl, device=DEV)
    _attention_parity(usv, q, k, v, wl.N, wl.k_per_head(), 64, 1)


@pytest.mark.parametrize("name", ["seq_99k", "seq_131k", "seq_193k"])
def test_sequence_length_sweep(usv, name):
    """The paper's speedup-vs-length points (about 99k / 131k / 193k tokens) at keep 5 %: selection
    in full (rows of 1560 / 2048 / 3023 scores: both selection kernels), attention on samples."""
    wl = ui.workload(name)
    q, k, v = ui.make_qkv(wl, device=DEV, layout="bhnd")
    _attention_parity(usv, q, k, v, wl.N, wl.k_per_head(), 24, 50 + wl.index)


@pytest.mark.parametrize("grid", [(64, 64, 64), (64, 17, 241)])
def test_longest_sequence_of_the_tensor_core_kernel_and_one_block_beyond(usv, grid):
    """4096 key blocks (262 144 tokens) is the longest sequence the tcgen05 attention kernel takes
    (its pairing plan keeps one bitmap row per query block in shared memory); with 4097 blocks the
    same call runs the exact online-softmax kernel instead.  One head, 40 key blocks kept: rows of
    4096 / 4097 scores through the selection kernel in full, attention on sampled query blocks."""
    wl = ui.Workload("longest", 40, 1, 1, 128, grid, (1,), k_fixed=40)
    assert wl.NB in (4096, 4097)
    q, k, v = ui.make_qkv(wl, device=DEV, layout="bhnd")
    _attention_parity(usv, q, k, v, wl.N, wl.k_per_head(), 6, 60 + wl.NB)


def test_wan_14b_720p(usv):
    wl = ui.workload("wan14b_720p")
    q, k, v = ui.make_qkv(wl, device=DEV)
    _attention_parity(usv, q, k, v, wl.N, wl.k_per_head(), 48, 2)


def _merge_pipeline(usv, wl, n_src_sample, n_qb, seed):
    z = ui.make_hidden(wl, DEV)
    w = ui.make_qkv_weight(wl, DEV)
    metric = (z @ w[:, wl.C:2 * wl.C]).reshape(wl.B, wl.N, wl.H, wl.d).contiguous()
    zm, plan = usv.token_merge(z, metric, wl.grid, wl.merge_part, wl.r, debug=True)
    torch.cuda.synchronize()
    pg = dict(dst_of=plan.dst_of.cpu().numpy(), pos=plan.pos.cpu().numpy(),
              u=plan.u.cpu().numpy(), jstar=plan.jstar.cpu().numpy())
    is_dst = oracle.destination_mask(wl.grid, wl.merge_part)
    src = np.nonzero(~is_dst)[0]
    rng = np.random.default_rng(seed)
    sample = np.sort(rng.choice(src, size=n_src_sample, replace=False))
    stats = check_merge_plan(pg, metric.cpu(), wl.grid, wl.merge_part, wl.r, src_sample=sample)
    print("merge plan:", stats)
    # merged values on three 64-channel slices (merging acts on every channel alike)
    Nm = wl.N - wl.r
    zc = z.cpu()
    got = bits(zm)
    worst = 0
    for c0 in (0, wl.C // 2, wl.C - 64):
        ref = oracle.round_to_bf16(oracle.merge_apply(zc[:, :, c0:c0 + 64].contiguous(), pg["dst_of"], pg["pos"], Nm))
        worst = max(worst, int(bf16_ulp_distance(got[:, :, c0:c0 + 64], ref).max()))
    assert worst <= 1
    # attention on the merged sequence
    N = wl.N_attn
    qkv = (zm @ w).reshape(wl.B, N, 3, wl.H, wl.d)
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    o = _attention_parity(usv, q, k, v, N, wl.k_per_head(), n_qb, seed)
    # unmerge of the attention output back to the full grid
    om = o.permute(0, 2, 1, 3).reshape(wl.B, N, wl.C)
    assert om.data_ptr() == o.data_ptr()
    y = usv.token_unmerge(om, plan.pos)
    torch.cuda.synchronize()
    assert y.shape == (wl.B, wl.N, wl.C)
    ref = oracle.unmerge(bits(om), pg["pos"])
    assert np.array_equal(bits(y), ref)


def test_wan_480p_merge50(usv):
    _merge_pipeline(usv, ui.workload("wan1.3b_480p_merge50"), 768, 48, 3)


def test_hunyuan_720p_mixed_keep_merge25(usv):
    _merge_pipeline(usv, ui.workload("hunyuan_720p"), 256, 48, 4)


@pytest.mark.parametrize("pct,n_qb", [(100, 6), (25, 16), (10, 24), (5, 24)])
def test_hunyuan_720p_uniform_keep(usv, pct, n_qb):
    """The keep-ratio sweep of the HunyuanVideo-shaped layer run one ratio at a time (every head
    keeps the same share of the key blocks), on the sequence left by the 25 % merge.  At keep
    100 % every block is selected and the oracle's sparse attention IS dense softmax attention
    (Eq. 4) over the 89 100 merged tokens."""
    wl = ui.workload("hunyuan_720p_keep%d" % pct)
    z = ui.make_hidden(wl, DEV)
    w = ui.make_qkv_weight(wl, DEV)
    metric = (z @ w[:, wl.C:2 * wl.C]).reshape(wl.B, wl.N, wl.H, wl.d).contiguous()
    zm, plan = usv.token_merge(z, metric, wl.grid, wl.merge_part, wl.r)
    del metric, z
    N = wl.N_attn
    qkv = (zm @ w).reshape(wl.B, N, 3, wl.H, wl.d)
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    kph = wl.k_per_head()
    assert kph == [(pct * wl.NB + 99) // 100] * wl.H
    o = _attention_parity(usv, q, k, v, N, kph, n_qb, 40 + pct, check_sel=(pct != 100))
    if pct == 100:
        sel = usv.select_blocks(usv.block_scores(q, k, N, N), kph)
        assert torch.equal(sel, torch.arange(wl.NB, dtype=torch.int32, device=DEV).expand_as(sel))
    assert torch.isfinite(o[:, :, :N].float()).all()
