"""Pins of the oracle's QK-norm + RoPE prologue against library routines and textbook properties."""
import numpy as np
import torch

import oracle


def _tables(N, d, base=10000.0, seed=None):
    """1-D rotary tables: angle[n, i] = n * base^(-2i/d) (or random angles)."""
    if seed is not None:
        ang = np.random.default_rng(seed).uniform(-np.pi, np.pi, size=(N, d // 2))
    else:
        ang = np.arange(N)[:, None] * base ** (-2.0 * np.arange(d // 2) / d)[None, :]
    return np.cos(ang), np.sin(ang), ang


def test_norm_step_matches_library_rms_norm():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((2, 3, 40, 16)) * rng.uniform(0.1, 10, size=(2, 3, 40, 1))
    g = rng.uniform(0.5, 1.5, 16)
    N = 33
    one, zero = np.ones((N, 8)), np.zeros((N, 8))                     # zero angle: the rotation is the identity
    y = oracle.qk_norm_rope(x, g, one, zero, N, 1e-6)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (16,), torch.from_numpy(g), 1e-6).numpy()
    np.testing.assert_allclose(y[:, :, :N], ref[:, :, :N], rtol=1e-13, atol=1e-13)
    assert (y[:, :, N:] == 0).all()
    # unit weight: every row comes out with RMS 1 (eps is negligible here); the input's scale drops out
    y1 = oracle.qk_norm_rope(x, np.ones(16), one, zero, N, 0.0)
    np.testing.assert_allclose(np.sqrt((y1[:, :, :N] ** 2).mean(-1)), 1.0, rtol=1e-13)
    np.testing.assert_allclose(oracle.qk_norm_rope(7.5 * x, np.ones(16), one, zero, N, 0.0), y1, rtol=1e-13, atol=1e-15)


def test_rotation_matches_complex_multiplication_and_hand_values():
    rng = np.random.default_rng(1)
    N, d = 21, 8
    x = rng.standard_normal((1, 2, N, d))
    cos, sin, ang = _tables(N, d, seed=5)
    # undo the norm by hand (g = row rms, eps = 0) so that only the rotation is left
    y = np.stack([oracle.qk_norm_rope(x[:, h:h + 1, n:n + 1], np.full(d, np.sqrt((x[0, h, n] ** 2).mean())),
                                      cos[n:n + 1], sin[n:n + 1], 1, 0.0)[0, 0, 0]
                  for h in range(2) for n in range(N)]).reshape(2, N, d)
    xc = torch.view_as_complex(torch.from_numpy(x[0]).reshape(2, N, d // 2, 2).contiguous())
    rot = torch.polar(torch.ones(N, d // 2, dtype=torch.float64), torch.from_numpy(ang))
    ref = torch.view_as_real(xc * rot).reshape(2, N, d).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-12)
    # a quarter turn sends the pair (a, b) to (-b, a); a rotation keeps each pair's length
    q = oracle.qk_norm_rope(np.array([[[[3.0, 4.0]]]]), np.array([np.sqrt(12.5)] * 2), np.zeros((1, 1)), np.ones((1, 1)), 1, 0.0)
    np.testing.assert_allclose(q[0, 0, 0], [-4.0, 3.0], atol=1e-14)
    pairs = lambda a: (a.reshape(*a.shape[:-1], -1, 2) ** 2).sum(-1)
    np.testing.assert_allclose(pairs(ref), pairs(x[0]), rtol=1e-12)


def test_relative_position_property():
    """With the 1-D tables angle = n * theta_i, <rope(q, m), rope(k, n)> depends on m - n only."""
    rng = np.random.default_rng(2)
    d, N = 16, 12
    cos, sin, _ = _tables(N, d)
    qv, kv = rng.standard_normal(d), rng.standard_normal(d)
    rq, rk = np.sqrt((qv ** 2).mean()), np.sqrt((kv ** 2).mean())
    Q = oracle.qk_norm_rope(np.tile(qv, (1, 1, N, 1)), np.full(d, rq), cos, sin, N, 0.0)[0, 0]
    K = oracle.qk_norm_rope(np.tile(kv, (1, 1, N, 1)), np.full(d, rk), cos, sin, N, 0.0)[0, 0]
    S = Q @ K.T
    for off in range(-4, 5):
        diag = np.diagonal(S, offset=off)
        np.testing.assert_allclose(diag, diag[0], rtol=1e-11, atol=1e-11)
    assert abs(S[0, 0] - qv @ kv) < 1e-11                                # offset 0: the plain dot product
    assert abs(S[3, 0] - S[0, 3]) > 1e-3                                  # ... and the sign of the offset matters
