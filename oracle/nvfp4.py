"""CPU oracle of the block-scaled 4-bit (NVFP4-style) quantiser for Q and K -- TEST INFRASTRUCTURE.

The paper's quantisation format is NVFP4 (its Quantization section and per-model appendix paragraphs) and it
cites the low-bit attention line of work for quantised QK^T; it prints no formula.  The format as read here,
fixed bit for bit so that CPU and GPU bytes can be compared (all scalar steps are fp32 round-to-nearest):

  element   e2m1: sign, 2 exponent bits, 1 mantissa bit; magnitudes {0, 0.5, 1, 1.5, 2, 3, 4, 6}; code = sign<<3 | index
  block     16 consecutive elements of the head dimension share one scale, an e4m3 value >= 0 (bias 7, no Inf,
            max 448, subnormals down to 2^-9)
  tensor    one fp32 scale g per (b, h)

  g    = amax(b,h) / (6 * 448)       over the tokens that exist; 1 if amax = 0
  sf   = e4m3( (amax(block) / 6) / g )                     round-to-nearest-even, saturating
  code = e2m1( x / (value(sf) * g) )                       round-to-nearest-even (even = mantissa bit 0), saturating
         at +-6; a block whose sf is 0 has all codes 0
  xhat = value(code) * value(sf) * g                        (the dequantised value, evaluated in fp64 here)

Two codes per byte, the even element in the low nibble.  Only tests, the smoke check and the bench's CPU legs
may import this module.
"""
from __future__ import annotations

import numpy as np

E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
BLOCK = 16


def e2m1_decode(code: np.ndarray) -> np.ndarray:
    code = np.asarray(code, np.uint8)
    return np.where(code & 8, -1.0, 1.0) * E2M1_VALUES[code & 7]


def e2m1_encode(y: np.ndarray) -> np.ndarray:
    """fp32 -> e2m1 code, round to nearest, ties to the code with mantissa bit 0, saturating; -0 keeps its sign.
    Written as the rounding rule on the grid's seven midpoints (not as a search)."""
    y = np.asarray(y, np.float32)
    a = np.abs(y).astype(np.float64)
    idx = np.zeros(y.shape, np.uint8)
    # midpoint between index i and i+1, and which side a tie goes to (the even index)
    for i, mid in enumerate([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]):
        up = (a > mid) if (i % 2 == 0) else (a >= mid)       # i even: tie stays at i; i odd: tie goes up to i+1
        idx = np.where(up, np.uint8(i + 1), idx)
    idx = np.where(np.isnan(a), np.uint8(7), idx)
    return (idx | (np.signbit(y).astype(np.uint8) << 3)).astype(np.uint8)


def _e4m3_tables():
    from . import e4m3_decode
    return np.array([e4m3_decode(c) for c in range(128)])      # codes 0..126 finite ascending, 127 NaN


def e4m3_encode_pos(u: np.ndarray) -> np.ndarray:
    """fp32 >= 0 -> e4m3 code (0..126), round to nearest even, saturating at 448."""
    u = np.asarray(u, np.float32).astype(np.float64)
    tab = _e4m3_tables()[:127]
    mid = (tab[:-1] + tab[1:]) / 2.0                    # exact in fp64
    lo = np.searchsorted(mid, u, side="left")           # number of midpoints strictly below u
    tie = (lo < mid.size) & (u == mid[np.minimum(lo, mid.size - 1)])
    code = np.where(tie & (lo % 2 == 1), lo + 1, lo)    # a tie between codes lo and lo+1 goes to the even one
    return np.minimum(code, 126).astype(np.uint8)


def quantize(x_bf16: np.ndarray, N: int):
    """x: [B,H,n_alloc,d] bf16 bits (uint16) or float.  Returns (codes u8 [B,H,n_alloc,d/2], sf u8 [B,H,n_alloc,d/16],
    g f32 [B,H]).  Rows >= N come back as zeros."""
    from . import bf16_to_f64
    x = bf16_to_f64(x_bf16) if x_bf16.dtype == np.uint16 else np.asarray(x_bf16, np.float64)
    xf = x.astype(np.float32)
    B, H, n_alloc, d = xf.shape
    assert d % BLOCK == 0
    tab = _e4m3_tables().astype(np.float32)
    codes = np.zeros((B, H, n_alloc, d // 2), np.uint8)
    sfs = np.zeros((B, H, n_alloc, d // BLOCK), np.uint8)
    g = np.ones((B, H), np.float32)
    f32 = np.float32
    for b in range(B):
        for h in range(H):
            v = xf[b, h, :N]
            amax = f32(np.abs(v).max()) if N > 0 else f32(0)
            gg = f32(amax / f32(6.0 * 448.0)) if amax > 0 else f32(1.0)
            g[b, h] = gg
            blk = v.reshape(N, d // BLOCK, BLOCK)
            a = np.abs(blk).max(axis=2).astype(np.float32)
            u = ((a / f32(6.0)).astype(np.float32) / gg).astype(np.float32)
            sf = e4m3_encode_pos(u)
            s = (tab[sf] * gg).astype(np.float32)                       # [N, d/16]
            with np.errstate(divide="ignore", invalid="ignore"):
                y = (blk / s[:, :, None]).astype(np.float32)
            c = e2m1_encode(y)
            c = np.where((tab[sf] == 0)[:, :, None], np.uint8(0), c).reshape(N, d)
            sfs[b, h, :N] = sf
            codes[b, h, :N] = c[:, 0::2] | (c[:, 1::2] << 4)
    return codes, sfs, g


def dequantize(codes: np.ndarray, sfs: np.ndarray, g: np.ndarray) -> np.ndarray:
    """-> float64 [B,H,n_alloc,d]: value(code) * value(sf) * g."""
    tab = _e4m3_tables()
    B, H, n_alloc, half = codes.shape
    c = np.empty((B, H, n_alloc, 2 * half), np.uint8)
    c[..., 0::2] = codes & 15
    c[..., 1::2] = codes >> 4
    s = np.repeat(tab[sfs], BLOCK, axis=3)
    return e2m1_decode(c) * s * g.astype(np.float64)[:, :, None, None]
