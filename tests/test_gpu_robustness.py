"""Checks that stand in for a memory sanitizer and a race detector, in forms that cannot fault
the device: canary-padded output buffers (nothing outside the documented extent of any output
is written), run-to-run bitwise determinism of the integer outputs and of the attention output,
and the bounded device-side wait reporting USV_ERR_TIMEOUT while the context stays usable."""
import numpy as np
import pytest
import torch

import usv_inputs as ui

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
USV_ERR_TIMEOUT = 5


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


def _canary(nbytes_payload, pad=4096):
    """uint8 buffer [pad | payload | pad] filled with 0xA5; returns (buffer, payload view)."""
    buf = torch.full((pad + nbytes_payload + pad,), 0xA5, dtype=torch.uint8, device=DEV)
    return buf, buf[pad:pad + nbytes_payload]


def _intact(buf, nbytes_payload, pad=4096):
    return bool((buf[:pad] == 0xA5).all().item()) and bool((buf[pad + nbytes_payload:] == 0xA5).all().item())


def test_bounded_wait_runs_out_and_the_context_survives(usv):
    assert usv.workspace_status() == 0
    usv.selftest_wait_timeout(limit_us=1000)
    assert usv.workspace_status() == USV_ERR_TIMEOUT
    assert b"0x80000000" in usv.lib().usv_last_error()
    assert usv.workspace_status() == 0                 # reported once, then cleared
    # the status word is sticky across later calls until it is read
    usv.selftest_wait_timeout(limit_us=500)
    wl = ui.workload("tiny")
    q, k, v = ui.make_qkv(wl, device=DEV)
    kph = wl.k_per_head()
    sel = usv.select_blocks(usv.block_scores(q, k), kph)
    o = usv.sparse_attn_fwd(q, k, v, sel, kph)
    assert usv.workspace_status() == USV_ERR_TIMEOUT
    # ... and the device still computes: same call again, clean status, same result
    o2 = usv.sparse_attn_fwd(q, k, v, sel, kph)
    assert usv.workspace_status() == 0
    assert torch.equal(o, o2)


@pytest.mark.parametrize("d,grid,B,H,kph", [(128, (3, 11, 17), 2, 3, [2, 9, 5]), (64, (2, 9, 13), 1, 2, [1, 4])])
def test_outputs_stay_inside_their_extents(usv, d, grid, B, H, kph):
    wl = ui.Workload("canary%d" % d, 300 + d, B, H, d, grid, (100,))
    q, k, v = ui.make_qkv(wl, device=DEV)
    N = wl.N                                   # 561 / 234 tokens: partial last block
    NB = (N + 63) // 64
    kmax = max(kph) + 3                        # a sel row wider than any k: the tail must be -1 only
    sbuf, spay = _canary(B * H * NB * NB * 4)
    scores = usv.block_scores(q, k, N, N, out=spay.view(torch.float32).view(B, H, NB, NB))
    lbuf, lpay = _canary(B * H * NB * kmax * 4)
    sel = usv.select_blocks(scores, kph, kmax=kmax, out=lpay.view(torch.int32).view(B, H, NB, kmax))
    selc = sel.cpu().numpy()
    for h in range(H):
        assert (selc[:, h, :, kph[h]:] == -1).all() and (selc[:, h, :, :kph[h]] >= 0).all()
    # o: rows of the padded last block at or beyond N belong to the caller
    Np = NB * 64
    obuf, opay = _canary(B * H * Np * d * 2)
    o_full = opay.view(torch.bfloat16).view(B, H, Np, d)
    fbuf, fpay = _canary(B * H * N * d * 4)
    ebuf, epay = _canary(B * H * N * 4)
    qp = torch.zeros((B, H, Np, d), dtype=torch.bfloat16, device=DEV); qp[:, :, :N] = q
    kp = torch.zeros_like(qp); kp[:, :, :N] = k
    vp = torch.zeros_like(qp); vp[:, :, :N] = v
    for impl in (0, 1):
        usv.sparse_attn_fwd(qp, kp, vp, sel, kph, N=N, out=o_full, return_f32=True, return_lse=True, impl=impl,
                            out_f32=fpay.view(torch.float32).view(B, H, N, d),
                            out_lse=epay.view(torch.float32).view(B, H, N))
        torch.cuda.synchronize()
        assert usv.workspace_status() == 0
        assert _intact(sbuf, spay.numel()) and _intact(lbuf, lpay.numel())
        assert _intact(obuf, opay.numel()) and _intact(fbuf, fpay.numel()) and _intact(ebuf, epay.numel())
        tail = o_full[:, :, N:].contiguous().view(torch.uint8)
        assert bool((tail == 0xA5).all().item()), "rows at or beyond N were written"


def test_merge_outputs_stay_inside_their_extents(usv):
    grid, part, r, C = (3, 5, 8), (1, 1, 2), 37, 72
    B, N = 2, 120
    g = torch.Generator().manual_seed(9)
    x = torch.randn(B, N, C, generator=g).to(torch.bfloat16).to(DEV)
    metric = torch.randn(B, N, 2, 64, generator=g).to(torch.bfloat16).to(DEV)
    mbuf, mpay = _canary(B * (N - r) * C * 2)
    xm, plan = usv.token_merge(x, metric, grid, part, r, out=mpay.view(torch.bfloat16).view(B, N - r, C))
    ybuf, ypay = _canary(B * N * C * 2)
    usv.token_unmerge(xm, plan.pos, out=ypay.view(torch.bfloat16).view(B, N, C))
    torch.cuda.synchronize()
    assert _intact(mbuf, mpay.numel()) and _intact(ybuf, ypay.numel())
    pos = plan.pos.cpu().numpy()
    assert pos.min() >= 0 and pos.max() == N - r - 1


def test_integer_outputs_and_attention_are_bitwise_reproducible(usv):
    """20 repeats of selection, merge plan and attention on the same inputs: no output may depend
    on the order in which CTAs or warps happen to run."""
    wl = ui.Workload("repeat", 77, 1, 4, 128, (6, 20, 26), (100,))          # 3120 tokens, 49 blocks
    q, k, v = ui.make_qkv(wl, device=DEV)
    N = wl.N - 5
    kph = [5, 12, 49, 1]
    z = ui.make_hidden(wl, DEV)
    metric = q.permute(0, 2, 1, 3).contiguous()                              # [B,N,H,d]
    first = None
    for _ in range(20):
        sel = usv.select_blocks(usv.block_scores(q, k, N, N), kph)
        o, lse = usv.sparse_attn_fwd(q, k, v, sel, kph, N=N, return_lse=True)
        zm, plan = usv.token_merge(z, metric, wl.grid, (1, 2, 2), 1000, debug=True)
        cur = [sel.clone(), o[:, :, :N].clone(), lse.clone(), plan.pos.clone(), plan.dst_of.clone(), plan.jstar.clone(), zm.clone()]
        if first is None:
            first = cur
        else:
            for a, b in zip(first, cur):
                assert torch.equal(a.view(torch.uint8) if a.dtype == torch.bfloat16 else a,
                                   b.view(torch.uint8) if b.dtype == torch.bfloat16 else b)
    assert usv.workspace_status() == 0
