"""Pins for the oracle's 4-bit block-scaled quantiser: the element grid, the rounding rule, the scale rule."""
import numpy as np
import torch

import oracle
from oracle import nvfp4


def test_all_sixteen_codes_round_trip_and_the_grid_is_e2m1():
    codes = np.arange(16, dtype=np.uint8)
    vals = nvfp4.e2m1_decode(codes)
    # e2m1 by its definition: exponent field e (bias 1), mantissa bit m: e = 0 -> m/2, else 2^(e-1) * (1 + m/2)
    ref = []
    for c in range(16):
        e, m = (c >> 1) & 3, c & 1
        mag = 0.5 * m if e == 0 else 2.0 ** (e - 1) * (1 + 0.5 * m)
        ref.append(-mag if c & 8 else mag)
    np.testing.assert_array_equal(vals, np.array(ref))
    back = nvfp4.e2m1_encode(vals.astype(np.float32))
    np.testing.assert_array_equal(back, codes)              # -0 keeps its sign bit: code 8


def test_every_finite_bf16_rounds_to_the_nearest_grid_value_ties_to_even():
    bits = np.arange(65536, dtype=np.uint32)
    x = (bits << 16).astype(np.uint32).view(np.float32)
    x = x[np.isfinite(x)]
    got = nvfp4.e2m1_decode(nvfp4.e2m1_encode(x))
    grid = nvfp4.E2M1_VALUES
    a = np.minimum(np.abs(x).astype(np.float64), 100.0)     # (saturating: anything beyond the grid is nearest to 6)
    dist = np.abs(a[:, None] - grid[None, :])
    best = dist.min(axis=1)
    cand = dist == best[:, None]                            # one or two nearest grid values
    even = (np.arange(8) % 2 == 0)[None, :]
    pick = np.where(cand.sum(1) == 2, np.argmax(cand & even, axis=1), np.argmax(cand, axis=1))
    ref = np.where(np.signbit(x), -1.0, 1.0) * grid[pick]
    np.testing.assert_array_equal(got, ref)
    assert nvfp4.e2m1_decode(nvfp4.e2m1_encode(np.float32([1e9, -1e9, 5.0, 2.5, 0.25, 0.75])))\
        .tolist() == [6.0, -6.0, 4.0, 2.0, 0.0, 1.0]


def test_scale_encoding_agrees_with_the_library_e4m3_cast():
    rng = np.random.default_rng(0)
    u = np.concatenate([rng.uniform(0, 500, 20000), rng.uniform(0, 0.05, 5000), [0.0, 448.0, 1e6, 2.0 ** -9, 2.0 ** -10]])
    u = u.astype(np.float32)
    ref = torch.from_numpy(np.minimum(u, 448.0)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    np.testing.assert_array_equal(nvfp4.e4m3_encode_pos(u), ref)
    # exact midpoints of the e4m3 grid: ties to the even code
    tab = np.array([oracle.e4m3_decode(c) for c in range(127)])
    mids = ((tab[:-1] + tab[1:]) / 2).astype(np.float32)
    exact = mids.astype(np.float64) == (tab[:-1] + tab[1:]) / 2
    got = nvfp4.e4m3_encode_pos(mids[exact])
    assert (got % 2 == 0).all()


def test_scale_rule_closed_forms_and_error_bound():
    d, N = 32, 5
    x = np.zeros((1, 1, 8, d))
    x[0, 0, 0, :16] = 6.0 * 448.0                           # the tensor's largest block: g = 1, sf = 448, codes +-6 -> exact
    x[0, 0, 0, 16:] = 3.0                                   # amax 3 -> sf = 0.5, elements 3.0 -> code 6.0
    x[0, 0, 1, :16] = np.linspace(-1.5, 1.5, 16)
    x[0, 0, 2] = 0.0                                        # an all-zero block: sf = 0, codes 0
    x[0, 0, 5:] = 123.0                                     # rows >= N do not exist
    codes, sfs, g = nvfp4.quantize(x, N)
    assert g[0, 0] == np.float32(1.0)
    assert oracle.e4m3_decode(int(sfs[0, 0, 0, 0])) == 448.0 and oracle.e4m3_decode(int(sfs[0, 0, 0, 1])) == 0.5
    xh = nvfp4.dequantize(codes, sfs, g)
    np.testing.assert_array_equal(xh[0, 0, 0], x[0, 0, 0])
    assert (codes[0, 0, 2] == 0).all() and (sfs[0, 0, 2] == 0).all() and (xh[0, 0, 2] == 0).all()
    assert (codes[0, 0, 5:] == 0).all() and (xh[0, 0, 5:] == 0).all()
    # block amax 1.5 -> sf = 0.25 exactly; the scaled grid's steps are 0.125 .. 0.5: every element within half the widest
    assert oracle.e4m3_decode(int(sfs[0, 0, 1, 0])) == 0.25
    assert np.abs(xh[0, 0, 1, :16] - x[0, 0, 1, :16]).max() <= 0.25 + 1e-12
    # random data: relative error of a block bounded by the grid's coarsest step (1 of 6 -> 1/6 of the block amax, plus the scale's rounding)
    rng = np.random.default_rng(1)
    y = rng.standard_normal((1, 2, 64, 64))
    c2, s2, g2 = nvfp4.quantize(y, 64)
    yh = nvfp4.dequantize(c2, s2, g2)
    blk = np.abs(y).reshape(1, 2, 64, 4, 16).max(-1, keepdims=True)
    err = np.abs(yh - y).reshape(1, 2, 64, 4, 16)
    assert (err <= blk * (1.0 / 6.0) * 1.07 + 1e-12).all()
    assert np.linalg.norm(yh - y) / np.linalg.norm(y) < 0.12
    # nibble order: even element in the low nibble
    z = np.zeros((1, 1, 1, 16)); z[0, 0, 0, 0] = 6.0; z[0, 0, 0, 1] = -3.0
    c3, _, _ = nvfp4.quantize(z, 1)
    assert c3[0, 0, 0, 0] == (7 | ((8 | 5) << 4))
