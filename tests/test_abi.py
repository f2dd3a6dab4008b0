"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared
symbol, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2512_05754_b200 import binding
    return binding.lib()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            txt = open(os.path.join(inc, fn)).read()
            txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
            names.update(re.findall(r"\b(usv_[a-z0-9_]+)\s*\(", txt))
    return sorted(names)


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert {"usv_block_scores", "usv_select_blocks", "usv_sparse_attn_fwd", "usv_token_merge",
            "usv_token_unmerge"} <= set(names)
    for n in names:
        assert hasattr(L, n), "libusv.so does not export %s" % n


def test_status_strings(L):
    assert L.usv_status_string(0) == b"ok"
    assert b"workspace" in L.usv_status_string(3)
    assert L.usv_build_info().startswith(b"usv-b200 sm_100a")


class S(ctypes.Structure):
    _fields_ = [("sb", ctypes.c_int64), ("sh", ctypes.c_int64), ("sn", ctypes.c_int64)]


def test_argument_validation_happens_on_the_host(L):
    p = ctypes.c_void_p(4096)         # a fake, aligned, never dereferenced device address
    s = S(128 * 128, 128, 128)
    ks = (ctypes.c_int32 * 2)(1, 1)
    z = ctypes.c_size_t(1 << 20)
    # unsupported head dim
    assert L.usv_block_scores(1, 2, 128, 128, 96, p, ctypes.byref(s), p, ctypes.byref(s), p, p, z, None) == 2
    assert b"d=96" in L.usv_last_error()
    # null pointer
    assert L.usv_block_scores(1, 2, 128, 128, 128, None, ctypes.byref(s), p, ctypes.byref(s), p, p, z, None) == 1
    # misaligned pointer / stride
    assert L.usv_block_scores(1, 2, 128, 128, 128, ctypes.c_void_p(4098), ctypes.byref(s), p, ctypes.byref(s), p, p, z, None) == 2
    bad = S(128 * 128, 128, 132)
    assert L.usv_block_scores(1, 2, 128, 128, 128, p, ctypes.byref(bad), p, ctypes.byref(s), p, p, z, None) == 2
    # workspace too small
    assert L.usv_block_scores(1, 2, 128, 128, 128, p, ctypes.byref(s), p, ctypes.byref(s), p, p, ctypes.c_size_t(16), None) == 3
    # k out of range, kmax too small
    bad_k = (ctypes.c_int32 * 2)(1, 9)
    assert L.usv_select_blocks(1, 2, 4, 8, p, bad_k, 9, p, None) == 1
    assert L.usv_select_blocks(1, 2, 4, 8, p, ks, 0, p, None) == 1
    assert L.usv_sparse_attn_fwd(1, 2, 128, 128, p, ctypes.byref(s), p, ctypes.byref(s), p, ctypes.byref(s),
                                 p, bad_k, 9, p, ctypes.byref(s), None, None, ctypes.c_float(0), 0, p, z, None) == 1
    # merge: r beyond the number of sources, grid mismatch, C not a multiple of 8
    assert L.usv_token_merge(1, 24, 64, p, 1, 64, p, 2, 3, 4, 1, 1, 2, 13, p, p, p, None, None, p, z, None) == 1
    assert L.usv_token_merge(1, 24, 64, p, 1, 64, p, 2, 3, 5, 1, 1, 2, 1, p, p, p, None, None, p, z, None) == 1
    assert L.usv_token_merge(1, 24, 60, p, 1, 64, p, 2, 3, 4, 1, 1, 2, 1, p, p, p, None, None, p, z, None) == 2
    assert L.usv_token_unmerge(1, 24, 30, 64, p, p, p, None) == 1
    # local merge: a negative window; cube order: empty grid, null output; forced own block: null scores
    assert L.usv_token_merge_local(1, 24, 64, p, 1, 64, p, 2, 3, 4, 1, 1, 2, 0, -1, 0, 3, p, p, p, None, None, p, z,
                                   None) == 1
    assert b"window" in L.usv_last_error()
    assert L.usv_cube_order(0, 3, 4, 4, 4, 4, p, None, None) == 1
    assert L.usv_cube_order(2, 3, 4, 4, 4, 4, None, None, None) == 1
    assert L.usv_force_own_block(1, 2, 4, 4, None, None) == 1
    # two-branch fusion: null scores; unsupported head width; null log-sum-exp; bad input-type flag
    assert L.usv_exclude_own_block(1, 2, 4, 4, None, None) == 1
    assert L.usv_attn_combine(1, 2, 128, 96, p, ctypes.byref(s), p, p, ctypes.byref(s), p, 0, p, ctypes.byref(s), None,
                              None, None) == 2
    assert L.usv_attn_combine(1, 2, 128, 128, p, ctypes.byref(s), None, p, ctypes.byref(s), p, 0, p, ctypes.byref(s),
                              None, None, None) == 1
    assert L.usv_attn_combine(1, 2, 128, 128, p, ctypes.byref(s), p, p, ctypes.byref(s), p, 7, p, ctypes.byref(s),
                              None, None, None) == 1
    # status helpers: null workspace
    assert L.usv_workspace_init(None, None) == 1
    assert L.usv_workspace_status(None, None) == 1
    assert L.usv_selftest_wait_timeout(p, 0, None) == 1


def test_workspace_sizes(L):
    L.usv_block_scores_workspace.restype = ctypes.c_size_t
    L.usv_token_merge_workspace.restype = ctypes.c_size_t
    # two fp32 pooled tensors [1,12,512,128]
    means = 2 * 12 * 512 * 128 * 4                             # pooled means of q and k, fp32
    planes = 12 * (512 + 512) * 128 * 3 * 2                    # three bf16 planes per operand
    header = 256                                               # status word at the head of every workspace
    assert L.usv_block_scores_workspace(1, 12, 32760, 32760, 128) == header + means + planes
    assert L.usv_block_scores_workspace(1, 2, 1024, 1024, 64) == header + 2 * 2 * 16 * 64 * 4   # d = 64: header + means
    assert L.usv_token_merge_workspace(1, 32760, 1536, 12, 128) >= 32760 * 128 * 4
