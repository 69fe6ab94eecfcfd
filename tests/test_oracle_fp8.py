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


# ------------------------------------------------------------------ K smoothing
def _offset_qkv(seed=7, B=1, H=2, N=200, n_alloc=256, d=16, offset=6.0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, H, n_alloc, d, generator=g).bfloat16()
    k = (torch.randn(B, H, n_alloc, d, generator=g) + offset * torch.randn(B, H, 1, d, generator=g)).bfloat16()
    v = torch.randn(B, H, n_alloc, d, generator=g).bfloat16()
    q[:, :, N:] = 0; k[:, :, N:] = 50.0; v[:, :, N:] = 0             # absent keys must not enter the mean
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    return (q, k, v), (bits(q), bits(k), bits(v))


def test_k_mean_closed_forms():
    (q, k, v), (qb, kb, vb) = _offset_qkv()
    N = 200
    m = oracle.k_mean(kb, N)
    assert m.shape == (1, 2, 16)
    np.testing.assert_allclose(m, k.double()[:, :, :N].mean(dim=2).numpy(), rtol=1e-13, atol=1e-13)
    # a constant key sequence is its own mean; an antisymmetric one has mean 0
    c = np.full((1, 1, 8, 4), 2.5)
    np.testing.assert_array_equal(oracle.k_mean(c, 6), np.full((1, 1, 4), 2.5))
    a = np.arange(-3, 4, dtype=np.float64).reshape(1, 1, 7, 1) * np.ones((1, 1, 1, 4))
    np.testing.assert_allclose(oracle.k_mean(a, 7), 0.0, atol=1e-15)


def test_smoothing_leaves_softmax_unchanged_and_shifts_lse():
    """Attention over (q, k - mean) equals attention over (q, k); lse moves by scale*<q, mean>."""
    (q, k, v), (qb, kb, vb) = _offset_qkv()
    N, block, scale = 200, 64, 0.25
    qf, kf, vf = (oracle.bf16_to_f64(x) for x in (qb, kb, vb))
    mean = oracle.k_mean(kb, N)
    ks = kf - mean[:, :, None, :]
    o0, l0 = oracle.dense_attn_rows(qf, kf, vf, N, block, scale)
    o1, l1 = oracle.dense_attn_rows(qf, ks, vf, N, block, scale)
    shift = oracle.lse_shift(qb, mean, N, scale)                      # [B,H,N]
    Nb = -(-N // block)
    for r in range(2 * Nb):
        bh, I = divmod(r, Nb)
        lo, hi = I * block, min((I + 1) * block, N)
        np.testing.assert_allclose(o1[r, : hi - lo], o0[r, : hi - lo], rtol=0, atol=1e-12)
        np.testing.assert_allclose(l1[r, : hi - lo] + shift[0, bh, lo:hi], l0[r, : hi - lo], rtol=0, atol=1e-11)
    # block routing sees the same thing: every row of the pooled scores moves by one constant
    s0 = oracle.block_scores(oracle.pool(qf, N, block), oracle.pool(kf, N, block), scale)
    s1 = oracle.block_scores(oracle.pool(qf, N, block), oracle.pool(ks, N, block), scale)
    dlt = s0 - s1
    np.testing.assert_allclose(dlt, dlt[..., :1] * np.ones_like(dlt), rtol=0, atol=1e-11)


def test_quantize_with_subtraction():
    (q, k, v), (qb, kb, vb) = _offset_qkv()
    N, block = 200, 64
    mean = oracle.k_mean(kb, N).astype(np.float32)
    # no subtraction and a zero subtraction are the same thing
    c0, s0 = oracle.quantize_e4m3(kb, N, block)
    cz, sz = oracle.quantize_e4m3(kb, N, block, sub=np.zeros_like(mean))
    np.testing.assert_array_equal(c0, cz); np.testing.assert_array_equal(s0, sz)
    # against the library cast of the same fp32 arithmetic
    cs, ss = oracle.quantize_e4m3(kb, N, block, sub=mean)
    kc = k.float() - torch.from_numpy(mean)[:, :, None, :]
    for h in range(2):
        for I in range(4):
            lo, hi = I * block, min((I + 1) * block, N)
            a = kc[0, h, lo:hi].abs().max()
            assert ss[0, h, I] == np.float32(a / 448.0)
            lib = (kc[0, h, lo:hi] / torch.tensor(ss[0, h, I])).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            np.testing.assert_array_equal(cs[0, h, lo:hi], lib)
    # what it is for: with a common offset in K the smoothed codes reproduce K far better
    kf = oracle.bf16_to_f64(kb)[:, :, :N]
    e_plain = np.abs(oracle.dequantize_e4m3(c0, s0, N, block)[:, :, :N] - kf).mean()
    e_smooth = np.abs(oracle.dequantize_e4m3(cs, ss, N, block)[:, :, :N] + mean[:, :, None, :].astype(np.float64) - kf).mean()
    assert e_smooth < 0.6 * e_plain, (e_smooth, e_plain)
