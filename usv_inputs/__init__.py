"""Seeded synthetic workloads shaped like video-DiT attention layers.

This module only manufactures INPUTS (and names the workload shapes).  It holds none of the
method's arithmetic and is the one piece of code that both the CPU oracle's tests and the CUDA
path's tests/benchmark may import.  The tensors stand in for the activations of Wan2.1 /
HunyuanVideo layers, which are not available offline.

Recipe, per tensor X, channel c, token at integer grid coordinates p = (t, y, x):

    X[p, c] = ( sum_{j=1..8} a_jc * sin(w_j . p + phi_jc) + 0.5 * n_pc ) * d^-0.25   -> bf16 (RNE)

a ~ N(0,1), phi ~ U(0, 2 pi), n ~ N(0,1) are independent per (tensor, j, c) / (tensor, p, c);
the eight wave vectors w_j ~ U(0, 0.5)^3 are shared by every tensor of one instance, which is
what gives queries and keys a common spatio-temporal structure.  All random numbers come from
a counter-based generator (splitmix64 of a mixed counter, Box-Muller for normals), so a value
depends only on (seed, tensor id, indices), not on chunking or device.
"""
import math
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

BS = 64  # tokens per attention block in every workload
_M64 = (1 << 64) - 1


def _s64(v):
    """Python int (mod 2^64) -> the signed int64 with the same bits."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLD = _s64(0x9E3779B97F4A7C15)
_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)


def _lsr(z, s):
    return (z >> s) & ((1 << (64 - s)) - 1)


def splitmix64(x):
    """One splitmix64 output step on an int64 tensor of counters (wrapping arithmetic)."""
    z = x + _GOLD
    z = (z ^ _lsr(z, 30)) * _C1
    z = (z ^ _lsr(z, 27)) * _C2
    return z ^ _lsr(z, 31)


def _key(seed, tensor_id, stream):
    """Scalar 64-bit stream key from (seed, tensor id, stream id), mixed on the host."""
    def mix(v):
        v = (v + 0x9E3779B97F4A7C15) & _M64
        v = ((v ^ (v >> 30)) * 0xBF58476D1CE4E5B9) & _M64
        v = ((v ^ (v >> 27)) * 0x94D049BB133111EB) & _M64
        return v ^ (v >> 31)
    k = mix(seed & _M64)
    k = mix(k ^ (tensor_id & _M64))
    k = mix(k ^ (stream & _M64))
    return _s64(k)


def uniform01(key, counters):
    """U(0,1) doubles (never 0 or 1) from int64 counters under a stream key."""
    z = splitmix64(counters ^ key)
    return (_lsr(z, 11).to(torch.float64) + 0.5) * (1.0 / (1 << 53))


def normal(key, counters):
    """N(0,1) doubles by Box-Muller from two decorrelated uniforms per counter."""
    u1 = uniform01(key, counters * 2)
    u2 = uniform01(key, counters * 2 + 1)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def wave_vectors(seed, device="cpu"):
    """The eight shared wave vectors w_j ~ U(0, 0.5)^3, fp64 [8,3]."""
    c = torch.arange(24, dtype=torch.int64, device=device)
    return (0.5 * uniform01(_key(seed, 0x77, 1), c)).reshape(8, 3)


def sin_field(seed, tensor_id, grid, channels, d_scale, device="cpu", n_rows=None,
              chunk_tokens=8192):
    """bf16 [n_rows, channels] field over the raster-ordered (t,y,x) grid; rows >= N are zero.

    d_scale is the head width d whose d^-0.25 scales the values."""
    T, Hh, W = grid
    N = T * Hh * W
    n_rows = N if n_rows is None else n_rows
    assert n_rows >= N
    dev = torch.device(device)
    out = torch.zeros((n_rows, channels), dtype=torch.bfloat16, device=dev)
    w = wave_vectors(seed, dev).to(torch.float32)                       # [8,3]
    jc = torch.arange(8 * channels, dtype=torch.int64, device=dev)
    a = normal(_key(seed, tensor_id, 2), jc).reshape(8, channels).to(torch.float32)
    phi = (2.0 * math.pi * uniform01(_key(seed, tensor_id, 3), jc)).reshape(8, channels)
    phi = phi.to(torch.float32)
    kn = _key(seed, tensor_id, 4)
    scale = float(d_scale) ** -0.25
    cidx = torch.arange(channels, dtype=torch.int64, device=dev)
    for lo in range(0, N, chunk_tokens):
        hi = min(N, lo + chunk_tokens)
        n = torch.arange(lo, hi, dtype=torch.int64, device=dev)
        p = torch.stack([n // (Hh * W), (n // W) % Hh, n % W], dim=1).to(torch.float32)  # [m,3]
        phase = p @ w.t()                                               # [m,8]
        acc = torch.zeros((hi - lo, channels), dtype=torch.float32, device=dev)
        for j in range(8):
            acc += a[j][None, :] * torch.sin(phase[:, j:j + 1] + phi[j][None, :])
        noise = normal(kn, n[:, None] * channels + cidx[None, :]).to(torch.float32)
        out[lo:hi] = ((acc + 0.5 * noise) * scale).to(torch.bfloat16)
    return out


def gaussian_weight(seed, tensor_id, rows, cols, device="cpu"):
    """bf16 [rows, cols] projection weight with N(0,1)/sqrt(rows) entries."""
    c = torch.arange(rows * cols, dtype=torch.int64, device=device)
    w = normal(_key(seed, tensor_id, 5), c).reshape(rows, cols) / math.sqrt(rows)
    return w.to(torch.bfloat16)


def keep_blocks(percent, nb):
    """Kept key blocks for an integer keep-percent of nb blocks: ceil(percent*nb/100), >= 1."""
    return max(1, (int(percent) * int(nb) + 99) // 100)


@dataclass
class Workload:
    """Shape of one synthetic attention-layer instance."""
    name: str
    index: int                      # position in the workload list; seed = 1234 + index
    B: int
    H: int
    d: int
    grid: Tuple[int, int, int]      # (T, Hh, W) token grid, raster order
    keep_percent: Tuple[int, ...]   # per head: keep_percent[h % len]
    k_fixed: Optional[int] = None   # explicit kept-block count (overrides keep_percent)
    merge_part: Optional[Tuple[int, int, int]] = None   # (st, sh, sw) or None = no merging
    merge_percent: int = 0          # r = floor(merge_percent * N / 100)
    note: str = ""

    @property
    def seed(self):
        return 1234 + self.index

    @property
    def N(self):
        return self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def r(self):
        return (self.merge_percent * self.N) // 100 if self.merge_part else 0

    @property
    def N_attn(self):
        """Sequence length seen by attention (after merging, if any)."""
        return self.N - self.r

    @property
    def NB(self):
        return (self.N_attn + BS - 1) // BS

    @property
    def C(self):
        return self.H * self.d

    def k_per_head(self):
        if self.k_fixed is not None:
            return [self.k_fixed] * self.H
        kp = self.keep_percent
        return [keep_blocks(kp[h % len(kp)], self.NB) for h in range(self.H)]


WORKLOADS = [
    Workload("tiny", 0, 1, 2, 64, (4, 16, 16), (25,), k_fixed=4,
             note="sanity instance; dense N x N oracle feasible"),
    Workload("wan1.3b_480p", 1, 1, 12, 128, (21, 30, 52), (10,),
             note="Wan2.1-1.3B 480p layer, 32760 tokens (+8 pad), 512 blocks, keep 10%"),
    Workload("wan1.3b_480p_merge50", 2, 1, 12, 128, (21, 30, 52), (10,),
             merge_part=(1, 1, 2), merge_percent=50,
             note="same grid, 50% bipartite merge of hidden states before attention"),
    Workload("wan14b_720p", 3, 1, 40, 128, (21, 45, 80), (5,),
             note="Wan 14B 720p-shaped layer, 75600 tokens, keep 5%"),
    Workload("hunyuan_720p", 4, 2, 24, 128, (33, 45, 80), (100, 25, 10, 5),
             merge_part=(1, 1, 2), merge_percent=25,
             note="HunyuanVideo 720p-shaped CFG pair, per-head keep sweep, 25% merge"),
    # Sequence-length sweep at the Wan2.1-1.3B head shape: the token counts of the paper's
    # speedup-vs-length study (about 99k / 131k / 193k tokens = 61 / 81 / 121 frames of a 60 x 104
    # latent grid before patchify), at its attention sparsity of 0.95 (keep 5 % of the key blocks).
    Workload("seq_99k", 5, 1, 12, 128, (16, 60, 104), (5,),
             note="length sweep, 99 840 tokens, 1560 blocks, keep 5%"),
    Workload("seq_131k", 6, 1, 12, 128, (21, 60, 104), (5,),
             note="length sweep, 131 040 tokens, 2048 blocks, keep 5%"),
    Workload("seq_193k", 7, 1, 12, 128, (31, 60, 104), (5,),
             note="length sweep, 193 440 tokens, 3023 blocks, keep 5%"),
    # The HunyuanVideo-shaped layer with one keep ratio on every head: the four points of its
    # keep-ratio sweep run one at a time (keep 100 % is dense attention over the merged sequence).
    Workload("hunyuan_720p_keep100", 8, 2, 24, 128, (33, 45, 80), (100,),
             merge_part=(1, 1, 2), merge_percent=25, note="uniform keep 100% (dense), 25% merge"),
    Workload("hunyuan_720p_keep25", 9, 2, 24, 128, (33, 45, 80), (25,),
             merge_part=(1, 1, 2), merge_percent=25, note="uniform keep 25%, 25% merge"),
    Workload("hunyuan_720p_keep10", 10, 2, 24, 128, (33, 45, 80), (10,),
             merge_part=(1, 1, 2), merge_percent=25, note="uniform keep 10%, 25% merge"),
    Workload("hunyuan_720p_keep5", 11, 2, 24, 128, (33, 45, 80), (5,),
             merge_part=(1, 1, 2), merge_percent=25, note="uniform keep 5%, 25% merge"),
]


def workload(name_or_index):
    for w in WORKLOADS:
        if w.name == name_or_index or w.index == name_or_index:
            return w
    raise KeyError(name_or_index)


def make_qkv(wl, device="cpu", layout="bhnd", N=None, grid=None):
    """Q, K, V for a workload without merging: bf16 views of logical shape [B,H,N,d].

    layout "bhnd": each is [B,H,N,d] contiguous.  layout "bnhd": memory is [B,N,H,d] and the
    returned tensors are permuted views (token stride H*d).  Channel index c = h*d + e."""
    grid = wl.grid if grid is None else grid
    out = []
    for tid in (1, 2, 3):
        per_b = [sin_field(wl.seed, 16 * b + tid, grid, wl.C, wl.d, device) for b in range(wl.B)]
        x = torch.stack(per_b, 0).reshape(wl.B, -1, wl.H, wl.d)          # [B,N,H,d]
        if layout == "bhnd":
            x = x.permute(0, 2, 1, 3).contiguous()
        else:
            x = x.permute(0, 2, 1, 3)
        out.append(x)
    return tuple(out)


def make_hidden(wl, device="cpu"):
    """Hidden states Z bf16 [B,N,C] for the merging workloads (C = H*d)."""
    per_b = [sin_field(wl.seed, 16 * b + 7, wl.grid, wl.C, wl.d, device) for b in range(wl.B)]
    return torch.stack(per_b, 0)


def make_qkv_weight(wl, device="cpu"):
    """Seeded projection C -> 3C, bf16 [C, 3C]; columns ordered (which, head, e)."""
    return gaussian_weight(wl.seed, 9, wl.C, 3 * wl.C, device)
