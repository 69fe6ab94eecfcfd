"""Pins for the oracle's e4m3 quantiser (O10)."""
import numpy as np
import torch

import oracle


def test_decode_matches_library_table():
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    mine = np.array([oracle.e4m3_decode(c) for c in range(256)])
    assert np.isnan(mine[[0x7f, 0xff]]).all() and np.isnan(ref[[0x7f, 0xff]]).all()
    ok = ~np.isnan(ref)
    np.testing.assert_array_equal(mine[ok], ref[ok])
    assert mine[0x7e] == 448.0 and mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6


def test_roundtrip_all_codes():
    for c in range(256):
        v = oracle.e4m3_decode(c)
        if np.isnan(v):
            continue
        assert oracle.e4m3_encode(v) == c or (v == 0 and oracle.e4m3_encode(v) in (0, 0x80))


def test_encode_all_bf16_patterns_vs_library_cast():
    """Every finite bf16 value: RNE cast against torch's float8_e4m3fn conversion where that is
    finite (|x| < 464), saturation to +-448 above."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    x = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float()
    fin = torch.isfinite(x)
    mine = np.array([oracle.e4m3_encode(float(v)) for v in x[fin].tolist()], np.uint8)
    xs = x[fin]
    lib = xs.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    # torch keeps the sign of zero results; so do we
    np.testing.assert_array_equal(mine, lib)
    big = xs.abs() >= 448
    assert set(mine[big.numpy()] & 0x7f) == {0x7e}


def test_midpoints_round_to_even():
    # between 1.0 (m=0) and 1.125 (m=1): midpoint 1.0625 -> even mantissa 0
    assert oracle.e4m3_encode(1.0625) == oracle.e4m3_encode(1.0)
    # between 1.125 and 1.25: midpoint 1.1875 -> even mantissa 2 (1.25)
    assert oracle.e4m3_decode(oracle.e4m3_encode(1.1875)) == 1.25
    # subnormal midpoint: 1.5 * 2^-9 -> 2 * 2^-9
    assert oracle.e4m3_decode(oracle.e4m3_encode(1.5 * 2 ** -9)) == 2 * 2 ** -9
    assert oracle.e4m3_decode(oracle.e4m3_encode(0.5 * 2 ** -9)) == 0.0


def test_quantize_blocks_scales_and_error_bound():
    B, H, N, d, block = 1, 2, 300, 16, 128
    n_alloc = 384
    g = torch.Generator().manual_seed(4)
    x = (torch.randn(B, H, n_alloc, d, generator=g) * 3).bfloat16()
    x[0, 1, 128:256] = 0                                  # an all-zero block -> scale 1
    x[:, :, N:] = 1000.0                                  # absent tokens must not set the scale
    bits = x.view(torch.int16).numpy().view(np.uint16)
    codes, scales = oracle.quantize_e4m3(bits, N, block)
    assert scales.shape == (B, H, 3) and scales.dtype == np.float32
    xf = x.float()
    for h in range(H):
        for I in range(3):
            lo, hi = I * block, min((I + 1) * block, N)
            a = xf[0, h, lo:hi].abs().max()
            exp = (a / 448.0) if a > 0 else torch.tensor(1.0)
            assert scales[0, h, I] == np.float32(exp)
            # codes against the library cast of the same fp32 quotient
            y = xf[0, h, lo:hi] / torch.tensor(scales[0, h, I])
            lib = y.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            np.testing.assert_array_equal(codes[0, h, lo:hi], lib)
    xhat = oracle.dequantize_e4m3(codes, scales, N, block)
    ref = xf.double().numpy()[:, :, :N]
    err = np.abs(xhat[:, :, :N] - ref)
    # normal range: relative error <= 2^-4; the whole block is bounded by absmax * 2^-4
    amax = np.repeat(scales.astype(np.float64) * 448, block, axis=-1)[:, :, :N, None]
    assert (err <= amax * 2.0 ** -4 + 1e-12).all()
    big = np.abs(ref) > amax * 2.0 ** -6
    assert (err[big] <= np.abs(ref[big]) * 2.0 ** -4 * (1 + 1e-6)).all()
    assert (xhat[:, :, N:] == 0).all()
