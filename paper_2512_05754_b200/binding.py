"""ctypes binding of libusv.so.  Same names as the C entry points, torch tensors in and out."""
import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

BLOCK = 64


class USVError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = "%s: %s (%s)" % (where, lib().usv_status_string(status).decode(),
                               lib().usv_last_error().decode())
        super().__init__(msg)


class _Strides(ctypes.Structure):
    _fields_ = [("sb", ctypes.c_int64), ("sh", ctypes.c_int64), ("sn", ctypes.c_int64)]


_lib = None


def lib_path():
    return _build.LIB


def lib():
    """Loads libusv.so (building it in-tree if it is missing and nvcc is available)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path):
        try:
            _build.build()
        except Exception as e:  # no silent fallback: the CUDA library is the product
            raise ImportError("libusv.so is not built and could not be built: %s" % e)
    L = ctypes.CDLL(path)
    L.usv_status_string.restype = ctypes.c_char_p
    L.usv_last_error.restype = ctypes.c_char_p
    L.usv_build_info.restype = ctypes.c_char_p
    L.usv_kernel_launches.restype = ctypes.c_ulonglong
    for name in ("usv_block_scores_workspace", "usv_sparse_attn_workspace",
                 "usv_token_merge_workspace", "usv_unmerge_map_workspace", "usv_merge_plan_cache_bytes"):
        getattr(L, name).restype = ctypes.c_size_t
    _lib = L
    return L


def build_info():
    return lib().usv_build_info().decode()


def kernel_launches():
    """Kernels the library has launched in this process so far."""
    return int(lib().usv_kernel_launches())


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream(device):
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _check(status, where):
    if status != 0:
        raise USVError(status, where)


def _view(t, name):
    if t.dim() != 4 or t.dtype != torch.bfloat16 or not t.is_cuda or t.stride(3) != 1:
        raise ValueError("%s must be a CUDA bf16 [B,H,N,d] view with a contiguous last axis" % name)
    return _Strides(t.stride(0), t.stride(1), t.stride(2))


_ws_cache = {}


WS_HEADER = 256


def _workspace(device, nbytes):
    """Grow-only scratch buffer per (device, stream).  Its header (status word) starts at zero
    and is carried over when the buffer grows, so that workspace_status() sees every call."""
    key = (device.index, torch.cuda.current_stream(device).cuda_stream)
    buf = _ws_cache.get(key)
    if buf is None or buf.numel() < nbytes:
        new = torch.empty(max(int(nbytes), WS_HEADER), dtype=torch.uint8, device=device)
        if buf is None:
            _check(lib().usv_workspace_init(_ptr(new), _stream(device)), "usv_workspace_init")
        else:
            new[:WS_HEADER].copy_(buf[:WS_HEADER])
        _ws_cache[key] = buf = new
    return buf


def _k_array(k_per_head, H):
    ks = [int(x) for x in k_per_head]
    if len(ks) != H:
        raise ValueError("k_per_head needs one entry per head")
    return (ctypes.c_int32 * H)(*ks), max(ks)


def block_scores(q, k, Nq=None, Nk=None, out=None):
    """scores[b,h,I,J] of the pooled 64-token blocks; fp32 [B,H,NBq,NBk]."""
    sq, sk = _view(q, "q"), _view(k, "k")
    B, H, nq, d = q.shape
    Nq = nq if Nq is None else int(Nq)
    Nk = k.shape[2] if Nk is None else int(Nk)
    NBq, NBk = (Nq + BLOCK - 1) // BLOCK, (Nk + BLOCK - 1) // BLOCK
    if out is None:
        out = torch.empty((B, H, NBq, NBk), dtype=torch.float32, device=q.device)
    L = lib()
    need = L.usv_block_scores_workspace(B, H, Nq, Nk, d)
    ws = _workspace(q.device, need)
    _check(L.usv_block_scores(B, H, Nq, Nk, d, _ptr(q), ctypes.byref(sq), _ptr(k),
                              ctypes.byref(sk), _ptr(out), _ptr(ws), ctypes.c_size_t(ws.numel()),
                              _stream(q.device)), "usv_block_scores")
    return out


def block_scores_noalloc(q, k, Nq=None, Nk=None, out=None):
    """block_scores for callers that must not allocate and have no scratch buffer to lend: the
    pooled means go to a fixed array inside the library (8 MiB per GPU), so only shapes whose
    scratch fits are accepted.  `out` should be passed by such callers (otherwise this wrapper
    allocates the result tensor through torch, which the C entry point itself never does).
    Calls on one device share the array: do not let two of them overlap on the GPU, and make the
    first call on a device outside any stream capture."""
    sq, sk = _view(q, "q"), _view(k, "k")
    B, H, nq, d = q.shape
    Nq = nq if Nq is None else int(Nq)
    Nk = k.shape[2] if Nk is None else int(Nk)
    NBq, NBk = (Nq + BLOCK - 1) // BLOCK, (Nk + BLOCK - 1) // BLOCK
    if out is None:
        out = torch.empty((B, H, NBq, NBk), dtype=torch.float32, device=q.device)
    _check(lib().usv_block_scores_noalloc(B, H, Nq, Nk, d, _ptr(q), ctypes.byref(sq), _ptr(k),
                                          ctypes.byref(sk), _ptr(out), _stream(q.device)),
           "usv_block_scores_noalloc")
    return out


def select_blocks(scores, k_per_head, kmax=None, out=None):
    """Top-k key blocks per (b,h,I), ascending, ties to the lowest index; int32 [B,H,NBq,kmax]."""
    if scores.dtype != torch.float32 or not scores.is_cuda or not scores.is_contiguous():
        raise ValueError("scores must be a contiguous CUDA fp32 tensor")
    B, H, NBq, NBk = scores.shape
    karr, kmx = _k_array(k_per_head, H)
    kmax = kmx if kmax is None else int(kmax)
    if out is None:
        out = torch.empty((B, H, NBq, kmax), dtype=torch.int32, device=scores.device)
    _check(lib().usv_select_blocks(B, H, NBq, NBk, _ptr(scores), karr, kmax, _ptr(out),
                                   _stream(scores.device)), "usv_select_blocks")
    return out


def sparse_attn_fwd(q, k, v, sel, k_per_head, N=None, scale=0.0, out=None, return_f32=False,
                    return_lse=False, impl=0, out_f32=None, out_lse=None):
    """Block-sparse attention forward.  Returns o (bf16, layout of q) and, if asked for, the
    un-rounded fp32 output [B,H,N,d] and the log-sum-exp [B,H,N] (written into out_f32 / out_lse
    when those contiguous fp32 tensors are given)."""
    sq, sk, sv = _view(q, "q"), _view(k, "k"), _view(v, "v")
    B, H, n, d = q.shape
    N = n if N is None else int(N)
    if sel.dtype != torch.int32 or not sel.is_contiguous() or not sel.is_cuda:
        raise ValueError("sel must be a contiguous CUDA int32 tensor")
    kmax = sel.shape[3]
    karr, _ = _k_array(k_per_head, H)
    if out is None:
        if q.is_contiguous():
            out = torch.empty_like(q)
        else:   # token-major memory [B,N,H,d], returned as a [B,H,N,d] view
            out = torch.empty((B, n, H, d), dtype=q.dtype, device=q.device).permute(0, 2, 1, 3)
    so = _view(out, "o")
    o32 = lse = None
    if return_f32:
        o32 = torch.empty((B, H, N, d), dtype=torch.float32, device=q.device) if out_f32 is None else out_f32
        if o32.dtype != torch.float32 or not o32.is_contiguous() or tuple(o32.shape) != (B, H, N, d):
            raise ValueError("out_f32 must be a contiguous fp32 [B,H,N,d] tensor")
    if return_lse:
        lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if out_lse is None else out_lse
        if lse.dtype != torch.float32 or not lse.is_contiguous() or tuple(lse.shape) != (B, H, N):
            raise ValueError("out_lse must be a contiguous fp32 [B,H,N] tensor")
    L = lib()
    need = L.usv_sparse_attn_workspace(B, H, N, d, kmax)
    ws = _workspace(q.device, need)
    _check(L.usv_sparse_attn_fwd(B, H, N, d, _ptr(q), ctypes.byref(sq), _ptr(k), ctypes.byref(sk),
                                 _ptr(v), ctypes.byref(sv), _ptr(sel), karr, kmax, _ptr(out),
                                 ctypes.byref(so), _ptr(o32), _ptr(lse), ctypes.c_float(scale),
                                 int(impl), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                 _stream(q.device)), "usv_sparse_attn_fwd")
    res = (out,)
    if return_f32:
        res += (o32,)
    if return_lse:
        res += (lse,)
    return res if len(res) > 1 else out


def workspace_status(device=None):
    """Synchronises the current stream and returns the status (0 = ok, 5 = a bounded device-side
    wait gave up in some call since the last query) of its workspace; a reported status is
    cleared."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    ws = _workspace(device, WS_HEADER)
    return lib().usv_workspace_status(_ptr(ws), _stream(device))


def selftest_wait_timeout(limit_us=1000, device=None):
    """Launches the library's bounded wait on a barrier nothing arrives at; workspace_status()
    reports USV_ERR_TIMEOUT afterwards (once)."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    ws = _workspace(device, WS_HEADER)
    _check(lib().usv_selftest_wait_timeout(_ptr(ws), ctypes.c_uint(int(limit_us)), _stream(device)),
           "usv_selftest_wait_timeout")


def sparse_attn_fallbacks(device=None):
    """Query blocks of the last sparse_attn_fwd on this stream that were recomputed exactly."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    ws = _workspace(device, WS_HEADER)
    n = ctypes.c_int(0)
    _check(lib().usv_sparse_attn_fallbacks(_ptr(ws), _stream(device), ctypes.byref(n)),
           "usv_sparse_attn_fallbacks")
    return n.value


@dataclass
class MergePlan:
    dst_of: torch.Tensor                 # int32 [B,N]
    pos: torch.Tensor                    # int32 [B,N]
    grid: tuple
    part: tuple
    r: int
    u: Optional[torch.Tensor] = None     # fp32 [B,N]
    jstar: Optional[torch.Tensor] = None  # int32 [B,N]
    cache: Optional[torch.Tensor] = None  # merged-source lists of the plan (merge_plan_cache)


def token_merge(x, metric, grid, part, r, plan=None, debug=False, window=None, out=None):
    """Merges x [B,N,C] (bf16).  With `metric` [B,N,Hm,dm] a new plan is computed; with
    metric=None the given `plan` is applied.  `window` = (wt, wh, ww) keeps the matching inside
    the partition blocks that near the source's own block (None: all destinations).
    Returns (x_merged [B,N-r,C], plan)."""
    if x.dim() != 3 or x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA bf16 [B,N,C] tensor")
    B, N, C = x.shape
    T, Hh, W = grid
    st, sh, sw = part
    dev = x.device
    if metric is None:
        if plan is None:
            raise ValueError("either metric or plan is needed")
        Hm = dm = 0
        u = js = None
    else:
        if metric.dim() != 4 or metric.dtype != torch.bfloat16 or not metric.is_contiguous():
            raise ValueError("metric must be a contiguous CUDA bf16 [B,N,Hm,dm] tensor")
        Hm, dm = metric.shape[2], metric.shape[3]
        plan = MergePlan(torch.empty((B, N), dtype=torch.int32, device=dev),
                         torch.empty((B, N), dtype=torch.int32, device=dev), tuple(grid),
                         tuple(part), int(r))
        if debug:
            plan.u = torch.empty((B, N), dtype=torch.float32, device=dev)
            plan.jstar = torch.empty((B, N), dtype=torch.int32, device=dev)
        u, js = plan.u, plan.jstar
    if out is None:
        out = torch.empty((B, max(N - r, 0), C), dtype=torch.bfloat16, device=dev)
    elif out.dtype != torch.bfloat16 or not out.is_contiguous() or tuple(out.shape) != (B, N - r, C):
        raise ValueError("out must be a contiguous bf16 [B,N-r,C] tensor")
    L = lib()
    need = L.usv_token_merge_workspace(B, N, C, Hm, dm if dm else 128)
    ws = _workspace(dev, need)
    if window is None:
        _check(L.usv_token_merge(B, N, C, _ptr(x), Hm, dm, _ptr(metric), T, Hh, W, st, sh, sw, int(r),
                                 _ptr(out), _ptr(plan.dst_of), _ptr(plan.pos), _ptr(u), _ptr(js),
                                 _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(dev)),
               "usv_token_merge")
    else:
        wt, wh, ww = (int(v) for v in window)
        _check(L.usv_token_merge_local(B, N, C, _ptr(x), Hm, dm, _ptr(metric), T, Hh, W, st, sh, sw, wt, wh, ww,
                                       int(r), _ptr(out), _ptr(plan.dst_of), _ptr(plan.pos), _ptr(u), _ptr(js),
                                       _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(dev)),
               "usv_token_merge_local")
    return out, plan


def token_unmerge(y_merged, pos, out=None):
    """y[b,n,:] = y_merged[b,pos[b,n],:]."""
    if (y_merged.dim() != 3 or y_merged.dtype != torch.bfloat16 or not y_merged.is_cuda
            or not y_merged.is_contiguous()):
        raise ValueError("y_merged must be a contiguous CUDA bf16 [B,Nm,C] tensor")
    B, Nm, C = y_merged.shape
    N = pos.shape[1]
    if out is None:
        out = torch.empty((B, N, C), dtype=torch.bfloat16, device=y_merged.device)
    _check(lib().usv_token_unmerge(B, N, Nm, C, _ptr(y_merged), _ptr(pos), _ptr(out),
                                   _stream(y_merged.device)), "usv_token_unmerge")
    return out


def attn_entropy(q, k, sel, k_per_head, lse, N=None, scale=0.0):
    """Key marginal [B,N] of the block-masked attention weights averaged over heads and queries,
    and its entropy normalised by log N [B].  `lse` is the log-sum-exp of sparse_attn_fwd for the
    same q, k, sel."""
    sq, sk = _view(q, "q"), _view(k, "k")
    B, H, n, d = q.shape
    N = n if N is None else int(N)
    if sel.dtype != torch.int32 or not sel.is_contiguous() or not sel.is_cuda:
        raise ValueError("sel must be a contiguous CUDA int32 tensor")
    if lse.dtype != torch.float32 or not lse.is_contiguous() or tuple(lse.shape) != (B, H, N):
        raise ValueError("lse must be a contiguous CUDA fp32 [B,H,N] tensor")
    karr, _ = _k_array(k_per_head, H)
    marg = torch.empty((B, N), dtype=torch.float32, device=q.device)
    ent = torch.empty((B,), dtype=torch.float32, device=q.device)
    ws = _workspace(q.device, WS_HEADER)
    _check(lib().usv_attn_entropy(B, H, N, d, _ptr(q), ctypes.byref(sq), _ptr(k), ctypes.byref(sk), _ptr(sel),
                                  karr, sel.shape[3], _ptr(lse), ctypes.c_float(scale), _ptr(marg), _ptr(ent),
                                  _ptr(ws), _stream(q.device)), "usv_attn_entropy")
    return marg, ent


def allocate_sparsity(entropy, gamma, rho_bar, rho_min, rho_max):
    """Per-layer ratios from per-layer entropies (host arithmetic): list of floats."""
    h = [float(x) for x in entropy]
    L = len(h)
    inp = (ctypes.c_float * L)(*h)
    out = (ctypes.c_float * L)()
    _check(lib().usv_allocate_sparsity(L, inp, ctypes.c_float(gamma), ctypes.c_float(rho_bar),
                                       ctypes.c_float(rho_min), ctypes.c_float(rho_max), out),
           "usv_allocate_sparsity")
    return list(out)


def cube_order(grid, cube=(4, 4, 4), device=None, want_inverse=True):
    """Token order in which the tokens of one local 3D cube are consecutive: returns (perm, inv)
    int32 [N] device tensors, perm[p] = raster index of the token at position p, inv its inverse
    (None unless wanted)."""
    T, Hh, W = (int(v) for v in grid)
    ct, ch, cw = (int(v) for v in cube)
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    n = max(T * Hh * W, 1)
    perm = torch.empty((n,), dtype=torch.int32, device=device)
    inv = torch.empty((n,), dtype=torch.int32, device=device) if want_inverse else None
    _check(lib().usv_cube_order(T, Hh, W, ct, ch, cw, _ptr(perm), _ptr(inv) if want_inverse else None,
                                _stream(device)), "usv_cube_order")
    return perm, inv


def permute_tokens(x, index):
    """y[b,p,:] = x[b,index[p],:] for a contiguous bf16 [B,N,C] tensor and an int32 [N] index (a
    permutation from cube_order): a row gather through usv_token_unmerge."""
    B = x.shape[0]
    pos = index.unsqueeze(0).expand(B, -1).contiguous()
    return token_unmerge(x, pos)


def force_own_block(scores):
    """In place: scores[b,h,I,I] = +inf, so that select_blocks keeps every query block's own block."""
    if scores.dtype != torch.float32 or not scores.is_contiguous() or not scores.is_cuda or scores.dim() != 4:
        raise ValueError("scores must be a contiguous CUDA fp32 [B,H,NBq,NBk] tensor")
    B, H, NBq, NBk = scores.shape
    _check(lib().usv_force_own_block(B, H, NBq, NBk, _ptr(scores), _stream(scores.device)), "usv_force_own_block")
    return scores


def exclude_own_block(scores):
    """In place: scores[b,h,I,I] = -inf, so that select_blocks never keeps a query block's own block
    (the long-range branch of the two-branch form)."""
    if scores.dtype != torch.float32 or not scores.is_contiguous() or not scores.is_cuda or scores.dim() != 4:
        raise ValueError("scores must be a contiguous CUDA fp32 [B,H,NBq,NBk] tensor")
    B, H, NBq, NBk = scores.shape
    _check(lib().usv_exclude_own_block(B, H, NBq, NBk, _ptr(scores), _stream(scores.device)), "usv_exclude_own_block")
    return scores


def attn_combine(o1, lse1, o2, lse2, out=None, return_f32=False, return_lse=False):
    """Fuses two attention branches over disjoint key sets by their softmax mass.  o1, o2: [B,H,N,d]
    views, both bf16 or both fp32; lse1, lse2: fp32 [B,H,N].  Returns o (bf16) [, o_f32] [, lse]."""
    if o1.dtype != o2.dtype or o1.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("o1 and o2 must both be bf16 or both be fp32")
    for t in (o1, o2):
        if t.dim() != 4 or not t.is_cuda or t.stride(3) != 1:
            raise ValueError("branch outputs must be CUDA [B,H,N,d] views with a contiguous last axis")
    B, H, N, d = o1.shape
    for l in (lse1, lse2):
        if l.dtype != torch.float32 or not l.is_contiguous() or tuple(l.shape) != (B, H, N):
            raise ValueError("lse must be a contiguous fp32 [B,H,N] tensor")
    s1 = _Strides(o1.stride(0), o1.stride(1), o1.stride(2))
    s2 = _Strides(o2.stride(0), o2.stride(1), o2.stride(2))
    if out is None:
        out = torch.empty((B, H, N, d), dtype=torch.bfloat16, device=o1.device)
    so = _view(out, "o")
    o32 = torch.empty((B, H, N, d), dtype=torch.float32, device=o1.device) if return_f32 else None
    lse = torch.empty((B, H, N), dtype=torch.float32, device=o1.device) if return_lse else None
    _check(lib().usv_attn_combine(B, H, N, d, _ptr(o1), ctypes.byref(s1), _ptr(lse1), _ptr(o2), ctypes.byref(s2),
                                  _ptr(lse2), 1 if o1.dtype == torch.float32 else 0, _ptr(out), ctypes.byref(so),
                                  _ptr(o32), _ptr(lse), _stream(o1.device)), "usv_attn_combine")
    res = (out,)
    if return_f32:
        res += (o32,)
    if return_lse:
        res += (lse,)
    return res if len(res) > 1 else out


def unmerge_map(pos, Nm):
    """Inverse of pos [B,N] (int32): (unmerge_off int32 [B,Nm+1], unmerge_idx int32 [B,N]), the
    original tokens grouped by the merged row they read back.  Built once per merge plan."""
    if pos.dtype != torch.int32 or not pos.is_contiguous() or not pos.is_cuda or pos.dim() != 2:
        raise ValueError("pos must be a contiguous CUDA int32 [B,N] tensor")
    B, N = pos.shape
    off = torch.empty((B, Nm + 1), dtype=torch.int32, device=pos.device)
    idx = torch.empty((B, N), dtype=torch.int32, device=pos.device)
    L = lib()
    ws = _workspace(pos.device, L.usv_unmerge_map_workspace(B, int(Nm)))
    _check(L.usv_unmerge_map(B, N, int(Nm), _ptr(pos), _ptr(off), _ptr(idx), _ptr(ws), ctypes.c_size_t(ws.numel()),
                             _stream(pos.device)), "usv_unmerge_map")
    return off, idx


def sparse_attn_fwd_unmerge(q, k, v, sel, k_per_head, umap, N_full, N=None, scale=0.0, out=None,
                            return_f32=False, return_lse=False):
    """sparse_attn_fwd on the merged sequence with the unmerge folded into its epilogue: returns
    y bf16 [B,N_full,H*d] (every original token holds the output row of its merged row) and, if
    asked for, the fp32 output / log-sum-exp in merged order.  umap = unmerge_map(plan.pos, N)."""
    sq, sk, sv = _view(q, "q"), _view(k, "k"), _view(v, "v")
    B, H, n, d = q.shape
    N = n if N is None else int(N)
    off, idx = umap
    if tuple(off.shape) != (B, N + 1) or tuple(idx.shape) != (B, int(N_full)):
        raise ValueError("unmerge map does not fit (B, N, N_full)")
    kmax = sel.shape[3]
    karr, _ = _k_array(k_per_head, H)
    if out is None:
        out = torch.empty((B, int(N_full), H * d), dtype=torch.bfloat16, device=q.device)
    scratch = torch.empty((B, n, H, d), dtype=q.dtype, device=q.device).permute(0, 2, 1, 3)
    so = _view(scratch, "o")
    o32 = torch.empty((B, H, N, d), dtype=torch.float32, device=q.device) if return_f32 else None
    lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if return_lse else None
    L = lib()
    ws = _workspace(q.device, L.usv_sparse_attn_workspace(B, H, N, d, kmax))
    _check(L.usv_sparse_attn_fwd_unmerge(B, H, N, d, _ptr(q), ctypes.byref(sq), _ptr(k), ctypes.byref(sk),
                                         _ptr(v), ctypes.byref(sv), _ptr(sel), karr, kmax, _ptr(scratch),
                                         ctypes.byref(so), _ptr(o32), _ptr(lse), ctypes.c_float(scale), _ptr(ws),
                                         ctypes.c_size_t(ws.numel()), int(N_full), _ptr(off), _ptr(idx), _ptr(out),
                                         _stream(q.device)), "usv_sparse_attn_fwd_unmerge")
    res = (out,)
    if return_f32:
        res += (o32,)
    if return_lse:
        res += (lse,)
    return res if len(res) > 1 else out


def merge_plan_cache(plan):
    """Builds (once) and returns the merged-source lists of a plan, kept on the plan object, so that
    token_merge_apply is the streaming merge kernel alone."""
    if plan.cache is None:
        B, N = plan.pos.shape
        T, Hh, W = plan.grid
        st, sh, sw = plan.part
        L = lib()
        nbytes = L.usv_merge_plan_cache_bytes(B, N)
        cache = torch.empty(int(nbytes), dtype=torch.uint8, device=plan.pos.device)
        _check(L.usv_merge_plan_cache(B, N, T, Hh, W, st, sh, sw, int(plan.r), _ptr(plan.dst_of), _ptr(plan.pos),
                                      _ptr(cache), ctypes.c_size_t(nbytes), _stream(plan.pos.device)),
               "usv_merge_plan_cache")
        plan.cache = cache
    return plan.cache


def token_merge_apply(x, plan, out=None):
    """Merges x [B,N,C] (bf16) with a stored plan through its cached lists; same result as
    token_merge(x, None, ..., plan=plan)."""
    if x.dim() != 3 or x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA bf16 [B,N,C] tensor")
    B, N, C = x.shape
    T, Hh, W = plan.grid
    st, sh, sw = plan.part
    cache = merge_plan_cache(plan)
    if out is None:
        out = torch.empty((B, N - plan.r, C), dtype=torch.bfloat16, device=x.device)
    _check(lib().usv_token_merge_apply(B, N, C, _ptr(x), T, Hh, W, st, sh, sw, int(plan.r), _ptr(cache), _ptr(out),
                                       _stream(x.device)), "usv_token_merge_apply")
    return out
