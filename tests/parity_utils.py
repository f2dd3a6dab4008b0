"""Helpers of the GPU-vs-oracle parity tests: admissibility of integer outputs inside the
near-tie band and error norms.  Everything here runs on the CPU with numpy."""
import numpy as np
import torch

import oracle

BAND = 1e-3          # relative near-tie band inside which integer outputs may legitimately differ


def bits(t):
    """CUDA/CPU bf16 tensor -> numpy uint16 bit patterns (contiguous copy)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def check_selection(sel_gpu, scores64, k_per_head):
    """Compares GPU block selections with the oracle's on fp64 scores.

    Rows must be identical unless the oracle's k-th and (k+1)-th scores are within BAND
    (relative); such rows must still be admissible: right size, ascending, and every block that
    differs from the oracle's choice scores inside the band around the cut.
    Returns (rows, ambiguous_rows, differing_rows)."""
    sel_gpu = np.asarray(sel_gpu)
    B, H, NBq, NBk = scores64.shape
    sel_ref, gap = oracle.select_blocks(scores64, k_per_head, kmax=sel_gpu.shape[3])
    differing = 0
    for h in range(H):
        k = int(k_per_head[h])
        g, r = sel_gpu[:, h, :, :k], sel_ref[:, h, :, :k]
        assert np.all(sel_gpu[:, h, :, k:] == -1), "tail must be -1"
        assert g.min() >= 0 and g.max() < NBk
        if k > 1:
            assert np.all(np.diff(g, axis=-1) > 0), "selection must be strictly ascending"
        bad = np.any(g != r, axis=-1)
        for b, i in zip(*np.nonzero(bad)):
            differing += 1
            assert gap[b, h, i] < BAND, (
                "selection differs outside the near-tie band: b=%d h=%d I=%d gap=%g" % (b, h, i, gap[b, h, i]))
            row = scores64[b, h, i]
            srt = np.sort(row)[::-1]
            tol = BAND * max(abs(srt[k - 1]), abs(srt[k]), 1e-30)
            only_gpu = np.setdiff1d(g[b, i], r[b, i])
            only_ref = np.setdiff1d(r[b, i], g[b, i])
            assert np.all(row[only_gpu] >= srt[k - 1] - tol) and np.all(row[only_ref] <= srt[k - 1] + tol)
    ambiguous = int((gap < BAND).sum())
    return B * H * NBq, ambiguous, differing


def attn_errors(o_gpu, o_ref):
    """(max abs error, relative L2 error) of two arrays of the same shape (fp64 math)."""
    a = np.asarray(o_gpu, dtype=np.float64)
    r = np.asarray(o_ref, dtype=np.float64)
    return float(np.abs(a - r).max()), float(np.linalg.norm(a - r) / max(np.linalg.norm(r), 1e-300))


def gather_qblocks(o, qb_list, N):
    """Rows of the query blocks in qb_list from an [B,H,N,d] tensor -> [n,64,d] (zero padded)."""
    o = o.detach().float().cpu().numpy() if isinstance(o, torch.Tensor) else o
    d = o.shape[-1]
    out = np.zeros((len(qb_list), 64) + ((d,) if o.ndim == 4 else ()), dtype=np.float64)
    for w, (b, h, i) in enumerate(qb_list):
        lo, hi = i * 64, min(N, i * 64 + 64)
        out[w, :hi - lo] = o[b, h, lo:hi]
    return out


def bf16_ulp_distance(a_bits, b_bits):
    """|a - b| in units of bf16 ulps for same-sign finite values (monotone integer mapping)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, 0x8000 - (x & 0x7fff) - 1, 0x8000 + x)
    return np.abs(key(a_bits) - key(b_bits))


def check_merge_plan(plan_gpu, metric_cpu, grid, part, r, src_sample=None, window=None):
    """Admissibility of a GPU merge plan against the oracle.  plan_gpu: dict of numpy arrays
    dst_of, pos, u, jstar ([B,N]).  Returns dict of counters."""
    mhat = oracle.merge_descriptors(metric_cpu)
    B, N, _ = mhat.shape
    is_dst = oracle.destination_mask(grid, part)
    src = np.nonzero(~is_dst)[0]
    if window is not None:
        assert src_sample is None
        sl, js, u, u2 = oracle.merge_match_local(mhat, grid, part, window)
        sl = sl.reshape(B, -1, 2); js = js.reshape(B, -1); u = u.reshape(B, -1); u2 = u2.reshape(B, -1)
        idx = sl[0, :, 1]
    elif src_sample is None:
        sl, js, u, u2 = oracle.merge_match(mhat, grid, part)
        sl = sl.reshape(B, -1, 2); js = js.reshape(B, -1); u = u.reshape(B, -1); u2 = u2.reshape(B, -1)
        idx = sl[0, :, 1]
    else:
        idx = np.asarray(src_sample, dtype=np.int32)
        pairs = np.stack([np.repeat(np.arange(B, dtype=np.int32), idx.size), np.tile(idx, B)], 1)
        _, js, u, u2 = oracle.merge_match(mhat, grid, part, pairs)
        js = js.reshape(B, -1); u = u.reshape(B, -1); u2 = u2.reshape(B, -1)
    stats = dict(sources=int(B * idx.size), jstar_ambiguous=0, jstar_differ=0, topr_band=0)
    gj, gu = plan_gpu["jstar"], plan_gpu["u"]
    assert np.all(gj[:, is_dst] == -1) and np.all(np.isnan(gu[:, is_dst]))
    for b in range(B):
        rel = (u[b] - u2[b]) / np.maximum(np.abs(u[b]), 1e-30)
        amb = rel < BAND
        stats["jstar_ambiguous"] += int(amb.sum())
        diff = gj[b, idx] != js[b]
        stats["jstar_differ"] += int(diff.sum())
        assert not np.any(diff & ~amb), "arg-max destination differs outside the near-tie band"
        for w in np.nonzero(diff)[0]:      # the GPU's choice must be a near-best destination
            c = float(mhat[b, idx[w]] @ mhat[b, gj[b, idx[w]]])
            assert c >= u[b, w] - BAND * abs(u[b, w])
        assert np.allclose(gu[b, idx], u[b], rtol=0, atol=2e-6), "cosine of the best match"
    # top-r: judged on the GPU's own u (fp32) against the oracle's threshold band
    dst_of, pos = plan_gpu["dst_of"], plan_gpu["pos"]
    for b in range(B):
        merged = dst_of[b] >= 0
        assert merged.sum() == r and not np.any(merged & is_dst)
        assert np.array_equal(dst_of[b][merged], gj[b][merged])
        if src_sample is None and 0 < r < src.size:
            srt = np.sort(u[b])[::-1]
            theta = srt[r - 1]
            uu = np.full(N, np.nan); uu[idx] = u[b]
            must = uu > theta * (1 + BAND) if theta > 0 else uu > theta + BAND
            mustnot = uu < theta * (1 - BAND) if theta > 0 else uu < theta - BAND
            assert np.all(merged[must]) and not np.any(merged[mustnot])
            inband = (~is_dst) & ~must & ~mustnot
            stats["topr_band"] += int(inband.sum())
            ref_merged, _ = oracle.merge_select(idx, u[b], r)
            stats.setdefault("topr_differ", 0)
            stats["topr_differ"] += int((merged[idx] != ref_merged).sum())
        # the selection step on its own: given the GPU's fp32 confidences, the merged set must be
        # exactly the oracle's top-r of those same values (ties to the lowest source index)
        ref_sel, _ = oracle.merge_select(src.astype(np.int32), gu[b, src].astype(np.float64), r)
        assert np.array_equal(merged[src], ref_sel), "top-r of the GPU's own confidences"
    pos_ref, nm = oracle.merge_positions(dst_of, grid, part)
    assert nm == N - r and np.array_equal(pos, pos_ref), "pos must follow from dst_of exactly"
    return stats
