"""ctypes front end of the fp64 CPU oracle (``usv_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing here is tuned, nothing here is used by the CUDA path.
bf16 tensors are passed as ``numpy.uint16`` bit patterns (or CPU ``torch.bfloat16`` tensors,
which are reinterpreted without copying the values through any float type).

Function -> passage of the paper (equations numbered in order of appearance):
  block_pool / block_scores / select_blocks : coarse "top-k cube selection" stage (Fig. 2 caption)
  dense_masked_attn / sparse_attn           : Sec. 3.2, Eq. 5
  merge_plan (+ its parts)                  : Sec. 3.3, Eq. 6-11, Eq. 14
  merge_apply / unmerge                     : Sec. 3.3, Eq. 12-13 / Eq. 15
  merge_match_local                         : Sec. 3.3, last paragraphs (matching kept inside
                                              neighbouring 3D blocks), the other reading of Eq. 8-9
  cube_order / select_blocks_local          : Fig. 2 caption (tokens grouped into local 3D cubes;
                                              attention in the own cube beside the top-k cubes)
  select_blocks_long_range / attn_combine   : Fig. 2 caption, the two-branch form: local cube
                                              attention and long-range top-k attention computed
                                              apart, their outputs fused.  The caption does not
                                              say how; the reading here weights each branch by
                                              its softmax mass (parity unpinned by the paper; the
                                              pins are the mathematics: it equals one attention
                                              over the union of the two disjoint key sets).
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "usv_oracle.c")
_LIB = os.path.join(_HERE, "libusv_oracle.so")
BS = 64

__all__ = [
    "BS", "build", "num_threads", "bf16_bits", "bf16_to_f64", "round_to_bf16", "block_pool",
    "block_scores", "select_blocks", "dense_masked_attn", "sparse_attn", "destination_mask",
    "merge_descriptors", "merge_match", "merge_select", "merge_positions", "merge_plan",
    "merge_apply", "unmerge", "all_query_blocks", "keep_count", "key_marginal", "entropy", "allocate",
    "cube_order", "select_blocks_local", "merge_match_local", "select_blocks_long_range", "attn_combine",
]


def build(force=False):
    """Compile the C oracle with gcc (plain -O2, OpenMP) into a shared object beside it."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.usvo_merge_positions.restype = ctypes.c_int
        _lib.usvo_num_threads.restype = ctypes.c_int
        _lib.usvo_entropy.restype = ctypes.c_double
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(x):
    return ctypes.c_int64(int(x))


def num_threads():
    return int(_L().usvo_num_threads())


def bf16_bits(x):
    """numpy uint16 view of a bf16 tensor (torch CPU bf16 tensor or uint16 ndarray)."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return x
    import torch
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.view(torch.int16).numpy().view(np.uint16)


def _strided(x):
    """(flat base array, element strides (sb,sh,sn)) of a 4-d bf16 view [B,H,N,d], d contiguous."""
    a = bf16_bits(x)
    assert a.ndim == 4 and a.strides[3] == 2
    st = tuple(s // 2 for s in a.strides[:3])
    # The C side indexes from element 0 of this view.
    return a, st


def bf16_to_f64(x):
    a = np.ascontiguousarray(bf16_bits(x))
    out = np.empty(a.shape, dtype=np.float64)
    _L().usvo_bf16_to_double(_p(a), _i64(a.size), _p(out))
    return out


def round_to_bf16(x):
    """fp64 ndarray -> bf16 bit patterns, round-to-nearest-even, single rounding."""
    a = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(a.shape, dtype=np.uint16)
    _L().usvo_round_to_bf16(_p(a), _i64(a.size), _p(out))
    return out


def keep_count(percent, nb):
    """Integer number of kept key blocks for an integer keep-percent: ceil(percent*nb/100)."""
    return max(1, (int(percent) * int(nb) + 99) // 100)


def block_pool(x, N):
    """x: bf16 [B,H,>=N,d] (any strides, d contiguous).  Returns fp64 [B,H,NB,d]."""
    a, (sb, sh, sn) = _strided(x)
    B, H, _, d = a.shape
    NB = (N + BS - 1) // BS
    out = np.empty((B, H, NB, d), dtype=np.float64)
    _L().usvo_block_pool(_p(a), B, H, int(N), d, _i64(sb), _i64(sh), _i64(sn), _p(out))
    return out


def block_scores(qbar, kbar):
    qbar = np.ascontiguousarray(qbar, dtype=np.float64)
    kbar = np.ascontiguousarray(kbar, dtype=np.float64)
    B, H, NBq, d = qbar.shape
    NBk = kbar.shape[2]
    s = np.empty((B, H, NBq, NBk), dtype=np.float64)
    _L().usvo_block_scores(_p(qbar), _p(kbar), B, H, NBq, NBk, d, _p(s))
    return s


def select_blocks(scores, k_per_head, kmax=None):
    """Returns (sel int32 [B,H,NBq,kmax] ascending with -1 tail, gap fp64 [B,H,NBq])."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    B, H, NBq, NBk = s.shape
    kph = np.ascontiguousarray(k_per_head, dtype=np.int32)
    assert kph.shape == (H,) and kph.min() >= 1 and kph.max() <= NBk
    kmax = int(kph.max()) if kmax is None else int(kmax)
    sel = np.empty((B, H, NBq, kmax), dtype=np.int32)
    gap = np.empty((B, H, NBq), dtype=np.float64)
    _L().usvo_select_blocks(_p(s), B, H, NBq, NBk, _p(kph), kmax, _p(sel), _p(gap))
    return sel, gap


def dense_masked_attn(q, k, v, N, sel, k_per_head, scale=None):
    """Literal N x N masked softmax attention (small N only).  q,k,v: bf16 [B,H,N,d] with the
    same strides.  Returns (o fp64 [B,H,N,d], rowsum fp64 [B,H,N])."""
    qa, st = _strided(q)
    ka, st_k = _strided(k)
    va, st_v = _strided(v)
    assert st == st_k == st_v
    B, H, _, d = qa.shape
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    kph = np.ascontiguousarray(k_per_head, dtype=np.int32)
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    o = np.empty((B, H, N, d), dtype=np.float64)
    rs = np.empty((B, H, N), dtype=np.float64)
    _L().usvo_dense_masked_attn(_p(qa), _p(ka), _p(va), B, H, int(N), d, _i64(st[0]), _i64(st[1]),
                                _i64(st[2]), _p(sel), _p(kph), sel.shape[3],
                                ctypes.c_double(scale), _p(o), _p(rs))
    return o, rs


def all_query_blocks(B, H, NB):
    b, h, i = np.meshgrid(np.arange(B), np.arange(H), np.arange(NB), indexing="ij")
    return np.ascontiguousarray(np.stack([b, h, i], axis=-1).reshape(-1, 3).astype(np.int32))


def sparse_attn(q, k, v, N, sel, k_per_head, scale=None, qb_list=None):
    """Masked attention restricted to the selected key blocks.

    q,k,v: bf16 [B,H,>=N,d], independent strides.  qb_list: int32 [n,3] of (b,h,I) or None for
    all query blocks in (b,h,I) order.  Returns (o fp64 [n,64,d], lse fp64 [n,64])."""
    qa, sq = _strided(q)
    ka, sk = _strided(k)
    va, sv = _strided(v)
    B, H, _, d = qa.shape
    NB = (N + BS - 1) // BS
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    assert sel.shape[:3] == (B, H, NB)
    kph = np.ascontiguousarray(k_per_head, dtype=np.int32)
    if qb_list is None:
        qb_list = all_query_blocks(B, H, NB)
    qb = np.ascontiguousarray(qb_list, dtype=np.int32)
    n = qb.shape[0]
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    o = np.empty((n, BS, d), dtype=np.float64)
    lse = np.empty((n, BS), dtype=np.float64)
    s3 = lambda s: (ctypes.c_int64 * 3)(*s)
    _L().usvo_sparse_attn(_p(qa), s3(sq), _p(ka), s3(sk), _p(va), s3(sv), B, H, int(N), d, _p(sel),
                          _p(kph), sel.shape[3], ctypes.c_double(scale), _p(qb), n, _p(o), _p(lse))
    return o, lse


# ------------------------------------------------------------------ token merging


def destination_mask(grid, part):
    T, Hh, W = grid
    st, sh, sw = part
    m = np.empty(T * Hh * W, dtype=np.uint8)
    _L().usvo_destination_mask(T, Hh, W, st, sh, sw, _p(m))
    return m.astype(bool)


def merge_descriptors(metric):
    """metric: bf16 [B,N,Hm,dm] contiguous -> unit descriptors fp64 [B,N,dm]."""
    a = np.ascontiguousarray(bf16_bits(metric))
    B, N, Hm, dm = a.shape
    out = np.empty((B, N, dm), dtype=np.float64)
    _L().usvo_merge_descriptors(_p(a), B, N, Hm, dm, _p(out))
    return out


def merge_match(mhat, grid, part, src_list=None):
    """Best destination of each source.  src_list: int32 [n,2] of (b,i) or None = all sources.
    Returns (src_list, jstar int32 [n], u fp64 [n], u2 fp64 [n])."""
    mhat = np.ascontiguousarray(mhat, dtype=np.float64)
    B, N, dm = mhat.shape
    T, Hh, W = grid
    st, sh, sw = part
    assert T * Hh * W == N
    if src_list is None:
        src = np.nonzero(~destination_mask(grid, part))[0].astype(np.int32)
        src_list = np.stack([np.repeat(np.arange(B, dtype=np.int32), src.size),
                             np.tile(src, B)], axis=1)
    sl = np.ascontiguousarray(src_list, dtype=np.int32)
    n = sl.shape[0]
    jstar = np.empty(n, dtype=np.int32)
    u = np.empty(n, dtype=np.float64)
    u2 = np.empty(n, dtype=np.float64)
    _L().usvo_merge_match(_p(mhat), B, N, dm, T, Hh, W, st, sh, sw, _p(sl), _i64(n), _p(jstar),
                          _p(u), _p(u2))
    return sl, jstar, u, u2


def merge_select(src_idx, u, r):
    """One batch element.  Returns (merged bool [n_src], theta (r-th, (r+1)-th largest u))."""
    src_idx = np.ascontiguousarray(src_idx, dtype=np.int32)
    u = np.ascontiguousarray(u, dtype=np.float64)
    n = src_idx.size
    assert 0 <= r <= n
    merged = np.empty(n, dtype=np.uint8)
    theta = np.empty(2, dtype=np.float64)
    _L().usvo_merge_select(_p(src_idx), _p(u), n, int(r), _p(merged), _p(theta))
    return merged.astype(bool), theta


def merge_positions(dst_of, grid, part):
    """dst_of int32 [B,N] (j* for merged sources, -1 otherwise) -> (pos int32 [B,N], Nm)."""
    d = np.ascontiguousarray(dst_of, dtype=np.int32)
    B, N = d.shape
    T, Hh, W = grid
    st, sh, sw = part
    pos = np.empty((B, N), dtype=np.int32)
    nm = _L().usvo_merge_positions(_p(d), B, T, Hh, W, st, sh, sw, _p(pos))
    assert nm >= 0, "batch elements disagree on the merged length"
    return pos, int(nm)


def merge_plan(metric, grid, part, r):
    """Whole plan (Eq. 6-11, 14) for every batch element.

    Returns dict: dst_of, pos [B,N] int32; jstar [B,N] int32 (-1 at destinations);
    u, u2 [B,N] fp64 (nan at destinations); theta [B,2]; Nm."""
    mhat = merge_descriptors(metric)
    B, N, _ = mhat.shape
    sl, js, u, u2 = merge_match(mhat, grid, part)
    n_src = sl.shape[0] // B
    assert r <= n_src, "r must not exceed the number of sources"
    jstar = np.full((B, N), -1, dtype=np.int32)
    uu = np.full((B, N), np.nan)
    uu2 = np.full((B, N), np.nan)
    dst_of = np.full((B, N), -1, dtype=np.int32)
    theta = np.empty((B, 2))
    for b in range(B):
        s = slice(b * n_src, (b + 1) * n_src)
        idx = sl[s, 1]
        jstar[b, idx] = js[s]
        uu[b, idx] = u[s]
        uu2[b, idx] = u2[s]
        merged, theta[b] = merge_select(idx, u[s], r)
        dst_of[b, idx[merged]] = js[s][merged]
    pos, nm = merge_positions(dst_of, grid, part)
    assert nm == N - r
    return dict(dst_of=dst_of, pos=pos, jstar=jstar, u=uu, u2=uu2, theta=theta, Nm=nm, mhat=mhat)


def merge_apply(x, dst_of, pos, Nm):
    """x: bf16 [B,N,C] -> fp64 [B,Nm,C] (mean aggregation, not yet rounded)."""
    a = np.ascontiguousarray(bf16_bits(x))
    B, N, C = a.shape
    d = np.ascontiguousarray(dst_of, dtype=np.int32)
    p = np.ascontiguousarray(pos, dtype=np.int32)
    out = np.empty((B, Nm, C), dtype=np.float64)
    _L().usvo_merge_apply(_p(a), B, N, C, _p(d), _p(p), int(Nm), _p(out))
    return out


def unmerge(y, pos):
    """y: bf16 [B,Nm,C] -> bf16 bits [B,N,C]."""
    a = np.ascontiguousarray(bf16_bits(y))
    B, Nm, C = a.shape
    p = np.ascontiguousarray(pos, dtype=np.int32)
    N = p.shape[1]
    out = np.empty((B, N, C), dtype=np.uint16)
    _L().usvo_unmerge(_p(a), B, N, C, Nm, _p(p), _p(out))
    return out


# ------------------------------------------------------------------ entropy-aware scheduler


def key_marginal(q, k, N, sel, k_per_head, scale=None):
    """Eq. 16 for the block-masked attention: fp64 [B,N], each row sums to one."""
    qa, sq = _strided(q)
    ka, sk = _strided(k)
    B, H, _, d = qa.shape
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    kph = np.ascontiguousarray(k_per_head, dtype=np.int32)
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    out = np.empty((B, int(N)), dtype=np.float64)
    s3 = lambda s: (ctypes.c_int64 * 3)(*s)
    _L().usvo_key_marginal(_p(qa), s3(sq), _p(ka), s3(sk), B, H, int(N), d, _p(sel), _p(kph), sel.shape[3],
                           ctypes.c_double(scale), _p(out))
    return out


def entropy(marg):
    """Eq. 17 per batch element: fp64 [B]."""
    m = np.ascontiguousarray(marg, dtype=np.float64)
    return np.array([_L().usvo_entropy(_p(m[b]), m.shape[1]) for b in range(m.shape[0])])


def allocate(h, gamma, rho_bar, rho_min, rho_max):
    """Eq. 18-19: per-layer ratios from per-layer entropies."""
    h = np.ascontiguousarray(h, dtype=np.float64)
    out = np.empty_like(h)
    _L().usvo_allocate(_p(h), h.shape[0], ctypes.c_double(gamma), ctypes.c_double(rho_bar),
                       ctypes.c_double(rho_min), ctypes.c_double(rho_max), _p(out))
    return out


def cube_order(grid, cube):
    """Token order in which the tokens of one local 3D cube are consecutive (Fig. 2 caption).

    grid = (T, Hh, W) in raster order, cube = (ct, ch, cw).  Cubes are taken in raster order of
    their cube coordinates, the tokens of a cube in raster order of their offsets inside it; a
    cube cut by the edge of the grid just holds fewer tokens (nothing is padded).  Returns
    (perm, inv): perm[p] = raster index of the token at position p of the cube order, inv its
    inverse.  Written as the definition: sort the tokens by (cube coordinate, offset)."""
    T, Hh, W = (int(v) for v in grid)
    ct, ch, cw = (int(v) for v in cube)
    t, y, x = np.meshgrid(np.arange(T), np.arange(Hh), np.arange(W), indexing="ij")
    t, y, x = t.ravel(), y.ravel(), x.ravel()
    # np.lexsort: last key is the primary one
    perm = np.lexsort((x % cw, y % ch, t % ct, x // cw, y // ch, t // ct)).astype(np.int32)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.size, dtype=np.int32)
    return perm, inv


def select_blocks_local(scores, k_per_head):
    """Selection with the local branch forced in: query block I always keeps key block I (its own
    cube), plus the k_h - 1 best of the other key blocks (ties -> lowest index); ascending, -1 tail.
    Returns (sel int32 [B,H,NBq,kmax], gap fp64 [B,H,NBq]): gap is the relative distance of the last
    kept and the first dropped score among the other blocks (inf when nothing is dropped or
    nothing else is kept)."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    B, H, NBq, NBk = s.shape
    kph = np.asarray(k_per_head, dtype=np.int64)
    kmax = int(kph.max())
    sel = np.full((B, H, NBq, kmax), -1, dtype=np.int32)
    gap = np.full((B, H, NBq), np.inf)
    for b in range(B):
        for h in range(H):
            k = int(kph[h])
            for i in range(NBq):
                own = i if i < NBk else None
                others = [j for j in range(NBk) if j != own]
                others.sort(key=lambda j: (-s[b, h, i, j], j))
                n_other = k - 1 if own is not None else k
                keep = others[:n_other] + ([own] if own is not None else [])
                sel[b, h, i, :k] = sorted(keep)
                if 0 < n_other < len(others):
                    a_, b_ = s[b, h, i, others[n_other - 1]], s[b, h, i, others[n_other]]
                    gap[b, h, i] = (a_ - b_) / max(abs(a_), abs(b_), 1e-30)
    return sel, gap


def select_blocks_long_range(scores, k_per_head):
    """Long-range branch of the two-branch form: for query block I the k_h best key blocks OTHER
    than block I (ties -> lowest index), ascending, -1 tail.  Where fewer than k_h other blocks
    exist all of them are kept.  Returns (sel, gap) like select_blocks_local."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    B, H, NBq, NBk = s.shape
    kph = np.asarray(k_per_head, dtype=np.int64)
    kmax = int(kph.max())
    sel = np.full((B, H, NBq, kmax), -1, dtype=np.int32)
    gap = np.full((B, H, NBq), np.inf)
    for b in range(B):
        for h in range(H):
            k = int(kph[h])
            for i in range(NBq):
                others = [j for j in range(NBk) if j != i]
                others.sort(key=lambda j: (-s[b, h, i, j], j))
                keep = others[:k]
                sel[b, h, i, :len(keep)] = sorted(keep)
                if 0 < k < len(others):
                    a_, b_ = s[b, h, i, others[k - 1]], s[b, h, i, others[k]]
                    gap[b, h, i] = (a_ - b_) / max(abs(a_), abs(b_), 1e-30)
    return sel, gap


def attn_combine(o1, lse1, o2, lse2):
    """Fusion of two attention branches over DISJOINT key sets (reading of the Fig. 2 caption):
    each branch's output is a softmax average over its own keys and lse its log-sum-exp, so the
    attention over both key sets together is the average of the two outputs weighted by
    exp(lse): o = (e^lse1 o1 + e^lse2 o2) / (e^lse1 + e^lse2), lse = log(e^lse1 + e^lse2).
    A branch without keys has lse = -inf and weight 0.  o*: [..., d], lse*: [...] -> (o, lse) fp64."""
    o1 = np.asarray(o1, dtype=np.float64)
    o2 = np.asarray(o2, dtype=np.float64)
    l1 = np.asarray(lse1, dtype=np.float64)
    l2 = np.asarray(lse2, dtype=np.float64)
    m = np.maximum(l1, l2)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    w1 = np.exp(l1 - m_safe)
    w2 = np.exp(l2 - m_safe)
    tot = w1 + w2
    with np.errstate(invalid="ignore", divide="ignore"):
        o = (w1[..., None] * o1 + w2[..., None] * o2) / tot[..., None]
        lse = m_safe + np.log(tot)
    o = np.where(tot[..., None] > 0, o, 0.0)
    return o, lse


def merge_match_local(mhat, grid, part, window):
    """Best destination of every source among the destinations of nearby partition blocks only
    (Sec. 3.3: sources and destinations confined to local 3D blocks; Eq. 8-9 with the arg-max
    over the blocks within `window` = (wt, wh, ww) blocks of the source's own block, per axis).

    The destination of a block is its first token in raster order.  Ties go to the lowest
    destination index.  Returns (src_list int32 [n,2] of (b,i), jstar int32 [n], u fp64 [n],
    u2 fp64 [n] = second-best similarity, -inf when there is no second candidate)."""
    mhat = np.ascontiguousarray(mhat, dtype=np.float64)
    B, N, dm = mhat.shape
    T, Hh, W = (int(v) for v in grid)
    st, sh, sw = (int(v) for v in part)
    wt, wh, ww = (int(v) for v in window)
    assert T * Hh * W == N and min(wt, wh, ww) >= 0
    nbt, nby, nbx = -(-T // st), -(-Hh // sh), -(-W // sw)
    src = np.nonzero(~destination_mask(grid, part))[0].astype(np.int32)
    t, rem = np.divmod(src, Hh * W)
    y, x = np.divmod(rem, W)
    bt, by, bx = t // st, y // sh, x // sw
    n = src.size
    jstar = np.full((B, n), -1, dtype=np.int32)
    u = np.full((B, n), -np.inf)
    u2 = np.full((B, n), -np.inf)
    # offsets in ascending order of the destination's raster index: a later candidate replaces
    # the best one only when strictly better
    for dt in range(-wt, wt + 1):
        for dy in range(-wh, wh + 1):
            for dx in range(-ww, ww + 1):
                ct, cy, cx = bt + dt, by + dy, bx + dx
                ok = (ct >= 0) & (ct < nbt) & (cy >= 0) & (cy < nby) & (cx >= 0) & (cx < nbx)
                j = ((ct * st) * Hh + cy * sh) * W + cx * sw
                w = np.nonzero(ok)[0]
                for b in range(B):
                    c = np.einsum("nd,nd->n", mhat[b, src[w]], mhat[b, j[w]])
                    better = c > u[b, w]
                    # the old best becomes the runner-up where it is beaten; otherwise c competes for runner-up
                    u2[b, w] = np.where(better, u[b, w], np.maximum(u2[b, w], c))
                    jstar[b, w] = np.where(better, j[w], jstar[b, w])
                    u[b, w] = np.where(better, c, u[b, w])
    sl = np.stack([np.repeat(np.arange(B, dtype=np.int32), n), np.tile(src, B)], axis=1)
    return sl, jstar.reshape(-1), u.reshape(-1), u2.reshape(-1)
