"""Seeded synthetic workloads shaped like the paper's Ovi- and LTX-class video/audio streams.

This module only *draws inputs*.  It holds none of the method's arithmetic (no attention, no
pooling, no top-k), so both the CUDA path and the CPU oracle may be fed from it.  The paper's own
measurements are on real Ovi / LTX-2.3 activations (Sec. 5.1), which need trained weights; the
tensors made here stand in for them by shape, value distribution and structure only.

Recipe (every tensor is ``[B, H, N, d]`` bf16, ``d`` contiguous):

* base: every element ~ N(0, 1), from a counter-based generator (splitmix64 of
  ``seed, tensor_id, flat_index`` -> two 24-bit uniforms -> Box-Muller), so a tensor's values do not
  depend on the order or chunking in which it is produced;
* smooth "3D-RoPE-like" structure (all but the tiny workload), added to the self-attention Q and K
  with the same field so that nearby positions have large q.k: for token (f, r, c) and channel j,
  axis ``j mod 3``, harmonic ``1 + (j // 3) mod 3``, a per-(head, channel) phase, amplitude
  ``a_pos * sqrt(2)``; the cross-attention video keys get the same field at half the amplitude;
* planted sound-source regions: a sign vector shared by all heads; cross-attention video keys inside
  a region get ``+2.0 * sign``, every audio query gets ``+0.25 * sign``, so audio queries concentrate
  on the regions (the situation the paper's Sec. 3 describes).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import torch

# tensor ids of the generator
TID_Q_SELF, TID_K_SELF, TID_V_SELF, TID_Q_AUDIO, TID_K_CROSS, TID_V_CROSS, TID_PHASE, TID_SIGN = range(8)

Region = Tuple[int, int, int, int, int, int]  # (f0, df, r0, dr, c0, dc)


@dataclass(frozen=True)
class Workload:
    """One attention layer's shapes.  Ratios are whole percentages; counts are derived by callers."""

    name: str
    B: int
    H: int
    d: int
    frames: int
    rows: int
    cols: int
    n_audio: int
    blk: int
    keep_pct: int
    protect_pct: int
    a_pos: float
    regions: Tuple[Region, ...] = field(default_factory=tuple)

    @property
    def n_video(self) -> int:
        return self.frames * self.rows * self.cols

    @property
    def n_blocks(self) -> int:
        return (self.n_video + self.blk - 1) // self.blk

    def with_ratios(self, keep_pct: int, protect_pct: int) -> "Workload":
        return Workload(self.name, self.B, self.H, self.d, self.frames, self.rows, self.cols,
                        self.n_audio, self.blk, keep_pct, protect_pct, self.a_pos, self.regions)


def _mid_regions() -> Tuple[Region, ...]:
    return tuple((8 * i, 6, (5 * i) % 16, 6, (7 * i) % 18, 6) for i in range(4))


def _ltx_regions() -> Tuple[Region, ...]:
    return tuple(((2 * i) % 14, 2, (5 * i) % 36, 12, (7 * i) % 50, 13) for i in range(8))


WORKLOADS: Dict[str, Workload] = {
    # batch 1, 2 heads, d 64, 4 x 8 x 8 video tokens, 32 audio tokens, block 64
    "tiny": Workload("tiny", 1, 2, 64, 4, 8, 8, 32, 64, 50, 10, 0.0, ((1, 2, 2, 4, 2, 4),)),
    # Ovi-class single layer
    "ovi": Workload("ovi", 1, 24, 128, 21, 30, 52, 256, 128, 25, 5, 1.0,
                    ((0, 5, 2, 8, 4, 10), (5, 5, 18, 8, 30, 10), (10, 5, 10, 8, 20, 10), (15, 5, 20, 8, 40, 10))),
    # mid-length sweep shape
    "mid": Workload("mid", 1, 24, 128, 31, 24, 24, 160, 128, 25, 5, 1.0, _mid_regions()),
    # LTX-class long sequence
    "ltx": Workload("ltx", 1, 32, 128, 16, 48, 64, 512, 128, 20, 5, 1.0, _ltx_regions()),
    # a small d=128 / block-128 case with a ragged tail block (N = 3*10*13 = 390 = 3*128 + 6)
    "small128": Workload("small128", 1, 3, 128, 3, 10, 13, 40, 128, 50, 10, 1.0, ((1, 1, 2, 4, 3, 5),)),
    # a medium d=128 case spanning many tiles with a ragged tail (N = 5*18*23 = 2070 = 16*128 + 22)
    "medium128": Workload("medium128", 2, 4, 128, 5, 18, 23, 72, 128, 25, 5, 1.0,
                          ((0, 2, 2, 6, 3, 8), (3, 2, 9, 6, 12, 8))),
}


# ----------------------------------------------------------------------------------------------
# counter-based generator (integer arithmetic only: identical on every device)
# ----------------------------------------------------------------------------------------------
def _i64(x: int) -> int:
    """Python int -> the int64 with the same low 64 bits."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _i64(0x9E3779B97F4A7C15)
_M1 = _i64(0xBF58476D1CE4E5B9)
_M2 = _i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    return (x >> k) & ((1 << (64 - k)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    z = x + _GOLD
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _key(seed: int, tensor_id: int) -> int:
    return _i64((seed * 0xD1342543DE82EF95 + (tensor_id + 1) * 0x9E3779B97F4A7C15) & ((1 << 64) - 1))


def _bits(seed: int, tensor_id: int, start: int, count: int, device) -> torch.Tensor:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _splitmix64(_splitmix64(idx ^ _key(seed, tensor_id)))


def normal_flat(seed: int, tensor_id: int, start: int, count: int, device) -> torch.Tensor:
    """``count`` N(0,1) fp32 values for flat indices ``start .. start+count-1`` of a tensor."""
    z = _bits(seed, tensor_id, start, count, device)
    u1 = (_lsr(z, 40).to(torch.float32) + 0.5) * (1.0 / 16777216.0)
    u2 = ((_lsr(z, 16) & 0xFFFFFF).to(torch.float32) + 0.5) * (1.0 / 16777216.0)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def uniform_flat(seed: int, tensor_id: int, start: int, count: int, device) -> torch.Tensor:
    z = _bits(seed, tensor_id, start, count, device)
    return (_lsr(z, 40).to(torch.float32) + 0.5) * (1.0 / 16777216.0)


# ----------------------------------------------------------------------------------------------
# structure
# ----------------------------------------------------------------------------------------------
def token_coords(w: Workload, device) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """(f, r, c) integer coordinates of every video token in raster order."""
    n = torch.arange(w.n_video, dtype=torch.int64, device=device)
    f = n // (w.rows * w.cols)
    r = (n // w.cols) % w.rows
    c = n % w.cols
    return f, r, c


def region_mask(w: Workload, device) -> torch.Tensor:
    """bool [N_v]: token lies inside a planted sound-source region."""
    f, r, c = token_coords(w, device)
    m = torch.zeros(w.n_video, dtype=torch.bool, device=device)
    for (f0, df, r0, dr, c0, dc) in w.regions:
        m |= (f >= f0) & (f < f0 + df) & (r >= r0) & (r < r0 + dr) & (c >= c0) & (c < c0 + dc)
    return m


def sign_vector(w: Workload, seed: int, device) -> torch.Tensor:
    """The shared +-1 direction of the planted regions, fp32 [d]."""
    u = uniform_flat(seed, TID_SIGN, 0, w.d, device)
    return torch.where(u < 0.5, -torch.ones_like(u), torch.ones_like(u))


def _smooth_field(w: Workload, seed: int, head: int, device) -> torch.Tensor:
    """fp32 [N_v, d] positional field of one head (amplitude 1; caller scales)."""
    f, r, c = token_coords(w, device)
    x = torch.stack([f.to(torch.float32) / w.frames, r.to(torch.float32) / w.rows,
                     c.to(torch.float32) / w.cols], dim=1)                      # [N, 3]
    j = torch.arange(w.d, device=device)
    axis = j % 3
    harm = (1 + (j // 3) % 3).to(torch.float32)
    phase = (2.0 * math.pi) * uniform_flat(seed, TID_PHASE, head * w.d, w.d, device)
    xa = x[:, axis]                                                             # [N, d]
    return math.sqrt(2.0) * torch.sin((2.0 * math.pi) * harm[None, :] * xa + phase[None, :])


def _tensor(w: Workload, seed: int, tid: int, n_tok: int, device,
            field_scale: float = 0.0, add_regions: float = 0.0, add_all: float = 0.0) -> torch.Tensor:
    out = torch.empty((w.B, w.H, n_tok, w.d), dtype=torch.bfloat16, device=device)
    per_head = n_tok * w.d
    sig = sign_vector(w, seed, device) if (add_regions or add_all) else None
    reg = region_mask(w, device) if add_regions else None
    for b in range(w.B):
        for h in range(w.H):
            x = normal_flat(seed, tid, (b * w.H + h) * per_head, per_head, device).view(n_tok, w.d)
            if field_scale:
                x = x + field_scale * _smooth_field(w, seed, h, device)
            if add_regions:
                x = x + add_regions * reg[:, None].to(torch.float32) * sig[None, :]
            if add_all:
                x = x + add_all * sig[None, :]
            out[b, h] = x.to(torch.bfloat16)
    return out


def make_self_qkv(w: Workload, seed: int = 0, device="cpu"):
    """Video self-attention Q, K, V: three bf16 ``[B, H, N_v, d]`` tensors."""
    q = _tensor(w, seed, TID_Q_SELF, w.n_video, device, field_scale=w.a_pos)
    k = _tensor(w, seed, TID_K_SELF, w.n_video, device, field_scale=w.a_pos)
    v = _tensor(w, seed, TID_V_SELF, w.n_video, device)
    return q, k, v


def make_cross_qkv(w: Workload, seed: int = 0, device="cpu"):
    """Audio->video cross-attention: audio Q ``[B,H,N_a,d]``, video K and V ``[B,H,N_v,d]`` (bf16)."""
    q = _tensor(w, seed, TID_Q_AUDIO, w.n_audio, device, add_all=0.25)
    k = _tensor(w, seed, TID_K_CROSS, w.n_video, device, field_scale=0.5 * w.a_pos, add_regions=2.0)
    v = _tensor(w, seed, TID_V_CROSS, w.n_video, device)
    return q, k, v


def loop_seed(step: int, layer: int) -> int:
    """Seed of layer ``layer`` at denoising step ``step`` in the multi-step loop workload."""
    return 1000 * step + layer


def all_workload_names() -> List[str]:
    return list(WORKLOADS)
