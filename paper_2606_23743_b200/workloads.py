"""Seeded synthetic Q/K/V shaped like video-DiT self-attention inputs.

This module holds input recipes only -- none of the method's arithmetic -- so both the
CUDA path's tests/bench and the CPU oracle's tests may draw their inputs from it.

The tensors stand in for the activations of a video diffusion transformer's spatiotemporal
self-attention (tokens of a T x H x W latent grid flattened with w fastest): i.i.d. N(0,1)
values plus a per-frame offset vector and a per-spatial-window offset vector added to both
Q and K, so that blocks of the same frame / same window score higher, which is the
structure block routing exploits.  Values are rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

SEED_BASE = 23743000


@dataclass(frozen=True)
class Workload:
    name: str
    cfg: int                 # seed offset
    B: int
    H: int
    d: int
    T: int
    Hg: int
    Wg: int
    block: int
    mode: int                # 0 top-k, 1 cumulative mass with cap
    k: int
    tau: float = 1.0
    win_t: int = -1          # forced neighbour half-widths (block-grid units); -1 = none
    win_s: int = -1
    sigma_f: float = 0.5     # std of the per-frame offset
    sigma_w: float = 0.0     # std of the per-window offset (0 = none)
    qk_mult: float = 1.0     # Q and K multiplied by this after the offsets
    fp8: bool = False

    @property
    def N(self) -> int:
        return self.T * self.Hg * self.Wg

    @property
    def Nb(self) -> int:
        return -(-self.N // self.block)

    @property
    def n_alloc(self) -> int:
        return self.Nb * self.block

    @property
    def R(self) -> int:
        return self.B * self.H * self.Nb

    @property
    def blocks_per_frame(self) -> int:
        per = self.Hg * self.Wg
        return per // self.block if per % self.block == 0 else 0

    @property
    def scale(self) -> float:
        return self.d ** -0.5


WORKLOADS = {
    "tiny": Workload("tiny", 1, B=1, H=2, d=64, T=4, Hg=16, Wg=16, block=64, mode=0, k=4),
    "medium": Workload("medium", 2, B=1, H=16, d=128, T=8, Hg=32, Wg=32, block=128, mode=0, k=16,
                       sigma_w=0.5),
    "large": Workload("large", 3, B=1, H=24, d=128, T=21, Hg=30, Wg=52, block=128, mode=1, k=40,
                      tau=0.9, sigma_w=0.5),
    "xl": Workload("xl", 4, B=2, H=32, d=128, T=31, Hg=32, Wg=48, block=128, mode=0, k=37,
                   win_t=1, win_s=1, sigma_w=0.5, qk_mult=1.5),
    "large_fp8": Workload("large_fp8", 5, B=1, H=24, d=128, T=21, Hg=30, Wg=52, block=128, mode=1,
                          k=40, tau=0.9, sigma_w=0.5, fp8=True),
    # paper-shaped second workload (its deployment preset: 64-token blocks, d = 128, about 10 % of the key
    # blocks kept); same tokens as "large", not a benchmark configuration
    "large_b64": Workload("large_b64", 7, B=1, H=24, d=128, T=21, Hg=30, Wg=52, block=64, mode=0, k=51,
                          sigma_w=0.5),
    # test-only variant of "large": stronger offsets so that the mass rule yields ragged rows
    "large_ragged": Workload("large_ragged", 6, B=1, H=24, d=128, T=21, Hg=30, Wg=52, block=128,
                             mode=1, k=40, tau=0.9, sigma_f=0.65, sigma_w=0.65),
}


def shrink(w: Workload, **kw) -> Workload:
    """A smaller copy of a workload (fewer heads / frames) with the same structure."""
    return replace(w, **kw)


def make_qkv(w: Workload, seed: int | None = None):
    """Returns bf16 CPU tensors q, k, v of shape [B, H, n_alloc, d]; rows >= N are zero."""
    g = torch.Generator(device="cpu")
    g.manual_seed(SEED_BASE + w.cfg if seed is None else seed)
    B, H, N, d = w.B, w.H, w.N, w.d
    q = torch.randn(B, H, N, d, generator=g, dtype=torch.float32)
    k = torch.randn(B, H, N, d, generator=g, dtype=torch.float32)
    v = torch.randn(B, H, N, d, generator=g, dtype=torch.float32)
    c = torch.randn(B, H, w.T, d, generator=g, dtype=torch.float32) * w.sigma_f
    tok = torch.arange(N)
    frame = tok // (w.Hg * w.Wg)
    off = c[:, :, frame, :]
    if w.sigma_w > 0:
        u = torch.randn(B, H, 16, d, generator=g, dtype=torch.float32) * w.sigma_w
        hh = (tok // w.Wg) % w.Hg
        ww = tok % w.Wg
        win = (4 * hh // w.Hg) * 4 + (4 * ww // w.Wg)
        off = off + u[:, :, win, :]
    q = (q + off) * w.qk_mult
    k = (k + off) * w.qk_mult
    out = []
    for x in (q, k, v):
        buf = torch.zeros(B, H, w.n_alloc, d, dtype=torch.bfloat16)
        buf[:, :, :N] = x.to(torch.bfloat16)
        out.append(buf)
    return tuple(out)


def bf16_bits(x: torch.Tensor):
    """bf16 CPU tensor -> numpy uint16 view of the same bits."""
    import numpy as np
    return x.contiguous().view(torch.int16).numpy().view(np.uint16)


def make_prologue_inputs(w: Workload, seed: int | None = None):
    """Inputs of the QK-norm + RoPE prologue for a workload's token grid: norm weights g_q, g_k [d] near 1,
    and rotary tables cos, sin [N, d/2] fp32 for a video's (frame, row, column) position -- the d/2
    frequencies split evenly over the three axes, angle = position * 10000^(-i / n) within an axis."""
    import math
    g = torch.Generator(device="cpu")
    g.manual_seed((SEED_BASE + w.cfg if seed is None else seed) + 7919)
    gq = 1.0 + 0.1 * torch.randn(w.d, generator=g, dtype=torch.float32)
    gk = 1.0 + 0.1 * torch.randn(w.d, generator=g, dtype=torch.float32)
    tok = torch.arange(w.N)
    pos = (tok // (w.Hg * w.Wg), (tok // w.Wg) % w.Hg, tok % w.Wg)
    half = w.d // 2
    bounds = [0, half // 3, 2 * (half // 3), half]
    ang = torch.zeros(w.N, half, dtype=torch.float64)
    for a in range(3):
        n = bounds[a + 1] - bounds[a]
        freq = torch.tensor([math.pow(10000.0, -i / n) for i in range(n)], dtype=torch.float64)
        ang[:, bounds[a]:bounds[a + 1]] = pos[a].double()[:, None] * freq[None, :]
    return gq, gk, torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
