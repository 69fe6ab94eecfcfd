"""Pins for the oracle's attention (O8/O9): brute force, a library routine, closed forms,
invariants.  None of these re-types the oracle's own loops."""
import numpy as np
import pytest
import torch

import oracle


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _brute_masked(q, k, v, N, block, scale, kept):
    """Explicit N x N boolean-mask softmax attention with numpy matrix algebra."""
    B, H, _, d = q.shape
    Nb = -(-N // block)
    out = np.zeros((B, H, N, d))
    lse = np.zeros((B, H, N))
    for b in range(B):
        for h in range(H):
            mask = np.zeros((N, N), bool)
            for I in range(Nb):
                for J in kept[(b * H + h) * Nb + I]:
                    mask[I * block:(I + 1) * block, J * block:(J + 1) * block] = True
            S = scale * q[b, h, :N] @ k[b, h, :N].T
            S = np.where(mask, S, -np.inf)
            m = S.max(-1, keepdims=True)
            P = np.exp(S - m)
            z = P.sum(-1, keepdims=True)
            out[b, h] = (P / z) @ v[b, h, :N]
            lse[b, h] = (m + np.log(z))[:, 0]
    return out, lse


def _csr(kept):
    row_ptr = np.zeros(len(kept) + 1, np.int32)
    row_ptr[1:] = np.cumsum([len(x) for x in kept])
    col = np.concatenate([np.asarray(x, np.int32) for x in kept])
    return row_ptr, col


def _unblock(o, B, H, N, block):
    """[R, block, d] -> [B,H,N,d] dropping the absent tail."""
    Nb = -(-N // block)
    d = o.shape[-1]
    return o.reshape(B, H, Nb * block, d)[:, :, :N]


@pytest.mark.parametrize("N,block,d", [(256, 64, 16), (200, 32, 8), (97, 16, 4)])
def test_brute_force_masked(N, block, d):
    B, H = 2, 2
    Nb = -(-N // block)
    n_alloc = Nb * block
    rng = np.random.default_rng(N)
    q, k, v = (_rand((B, H, n_alloc, d), s) for s in (1, 2, 3))
    # garbage in the absent tail must not matter
    q[:, :, N:] = 77.0; k[:, :, N:] = 55.0; v[:, :, N:] = -99.0
    kept = [sorted(rng.choice(Nb, size=rng.integers(1, Nb + 1), replace=False).tolist())
            for _ in range(B * H * Nb)]
    row_ptr, col = _csr(kept)
    o, lse = oracle.attn_rows(q, k, v, N, block, 0.37, row_ptr, col)
    ref, ref_lse = _brute_masked(q, k, v, N, block, 0.37, kept)
    np.testing.assert_allclose(_unblock(o, B, H, N, block), ref, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse.reshape(B, H, -1)[:, :, :N], ref_lse, rtol=1e-12, atol=1e-12)
    # absent query rows are never written
    if N % block:
        assert np.isnan(o.reshape(B, H, n_alloc, d)[:, :, N:]).all()


def test_library_sdpa_block_mask():
    """torch's scaled_dot_product_attention in float64 with a boolean block mask."""
    B, H, N, d, block = 1, 2, 1024, 64, 64
    Nb = N // block
    rng = np.random.default_rng(5)
    q, k, v = (_rand((B, H, N, d), s) for s in (11, 12, 13))
    kept = [sorted(rng.choice(Nb, size=4, replace=False).tolist()) for _ in range(B * H * Nb)]
    row_ptr, col = _csr(kept)
    o, _ = oracle.attn_rows(q, k, v, N, block, d ** -0.5, row_ptr, col)
    mask = torch.zeros(B, H, N, N, dtype=torch.bool)
    for r, ks in enumerate(kept):
        bh, I = divmod(r, Nb)
        for J in ks:
            mask[bh // H, bh % H, I * block:(I + 1) * block, J * block:(J + 1) * block] = True
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), attn_mask=mask)
    np.testing.assert_allclose(_unblock(o, B, H, N, block), ref.numpy(), rtol=1e-10, atol=1e-12)


def test_library_sdpa_dense_and_bf16_inputs():
    """Dense oracle vs torch SDPA (float64) on bf16-valued inputs given as bit patterns."""
    B, H, N, d, block = 1, 2, 200, 32, 64
    n_alloc = 256
    t = [torch.randn(B, H, n_alloc, d, generator=torch.Generator().manual_seed(s)).bfloat16()
         for s in (1, 2, 3)]
    bits = [x.view(torch.int16).numpy().view(np.uint16) for x in t]
    o, _ = oracle.dense_attn_rows(*bits, N, block, d ** -0.5)
    q, k, v = (x.double()[:, :, :N] for x in t)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v)
    np.testing.assert_allclose(_unblock(o, B, H, N, block), ref.numpy(), rtol=1e-10, atol=1e-12)
    # widening helper is exact
    np.testing.assert_array_equal(oracle.bf16_to_f64(bits[0]), t[0].double().numpy())


@pytest.mark.parametrize("N,block", [(1000, 64), (256, 64), (130, 128)])
def test_keep_all_equals_dense(N, block):
    """Keep-ratio 1.0 must be dense attention, including a ragged last block."""
    B, H, d = 1, 2, 16
    Nb = -(-N // block)
    q, k, v = (_rand((B, H, Nb * block, d), s) for s in (21, 22, 23))
    kept = [list(range(Nb))] * (B * H * Nb)
    row_ptr, col = _csr(kept)
    o1, l1 = oracle.attn_rows(q, k, v, N, block, 0.25, row_ptr, col)
    o2, l2 = oracle.dense_attn_rows(q, k, v, N, block, 0.25)
    ok = ~np.isnan(o2)
    assert (np.isnan(o1) == np.isnan(o2)).all()
    np.testing.assert_allclose(o1[ok], o2[ok], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(l1[~np.isnan(l2)], l2[~np.isnan(l2)], rtol=1e-13)


def test_rows_sum_to_one_and_convex_hull():
    B, H, N, d, block = 1, 3, 512, 8, 64
    Nb = N // block
    rng = np.random.default_rng(9)
    q, k, v = (_rand((B, H, N, d), s) for s in (31, 32, 33))
    kept = [sorted(rng.choice(Nb, size=3, replace=False).tolist()) for _ in range(B * H * Nb)]
    row_ptr, col = _csr(kept)
    scale = 0.5
    o, lse = oracle.attn_rows(q, k, v, N, block, scale, row_ptr, col)
    o = _unblock(o, B, H, N, block)
    lse = lse.reshape(B, H, N)
    for r, ks in enumerate(kept):
        h, I = divmod(r, Nb)
        cols = np.concatenate([np.arange(J * block, (J + 1) * block) for J in ks])
        rows = slice(I * block, (I + 1) * block)
        S = scale * q[0, h, rows] @ k[0, h, cols].T
        w = np.exp(S - lse[0, h, rows, None])
        np.testing.assert_allclose(w.sum(-1), 1.0, rtol=1e-12)       # weights sum to one
        vmin, vmax = v[0, h, cols].min(0), v[0, h, cols].max(0)       # coordinate-wise hull
        assert (o[0, h, rows] >= vmin - 1e-12).all() and (o[0, h, rows] <= vmax + 1e-12).all()


def test_closed_forms():
    B, H, N, d, block = 1, 1, 192, 8, 64
    q = _rand((B, H, N, d), 41)
    k = _rand((B, H, N, d), 42)
    v = _rand((B, H, N, d), 43)
    kept = [[0, 2], [1], [0, 1, 2]]
    row_ptr, col = _csr(kept)
    # V constant -> O is that constant
    vc = np.broadcast_to(np.arange(d, dtype=np.float64), v.shape).copy()
    o, _ = oracle.attn_rows(q, k, vc, N, block, 1.0, row_ptr, col)
    np.testing.assert_allclose(o, np.broadcast_to(np.arange(d), o.shape), rtol=1e-13)
    # all K rows equal -> O is the plain mean of V over the kept keys, lse = logit + log n
    ke = np.broadcast_to(k[0, 0, 0], k.shape).copy()
    o, lse = oracle.attn_rows(q, ke, v, N, block, 0.3, row_ptr, col)
    for I, ks in enumerate(kept):
        cols = np.concatenate([np.arange(J * block, (J + 1) * block) for J in ks])
        np.testing.assert_allclose(o[I], np.broadcast_to(v[0, 0, cols].mean(0), (block, d)), rtol=1e-12)
        np.testing.assert_allclose(lse[I], 0.3 * q[0, 0, I * block:(I + 1) * block] @ k[0, 0, 0] + np.log(len(cols)), rtol=1e-12)
    # one key far above the others -> O is that key's V row
    q1 = np.zeros_like(q); q1[..., 0] = 1.0
    k1 = np.zeros_like(k); k1[0, 0, 70, 0] = 60.0
    o, _ = oracle.attn_rows(q1, k1, v, N, block, 1.0, row_ptr, col)
    np.testing.assert_allclose(o[1], np.broadcast_to(v[0, 0, 70], (block, d)), rtol=0, atol=1e-12)
    # ... and a transposed-operand mistake (Q K^T vs K Q^T) would show here: asymmetric q, k
    q2 = np.zeros_like(q); q2[0, 0, 5, 1] = 50.0
    k2 = np.zeros_like(k); k2[0, 0, 9, 1] = 1.0
    o, _ = oracle.attn_rows(q2, k2, v, N, block, 1.0, *_csr([[0], [1], [2]]))
    np.testing.assert_allclose(o[0, 5], v[0, 0, 9], atol=1e-12)
    np.testing.assert_allclose(o[0, 6], v[0, 0, :64].mean(0), atol=1e-12)


def test_row_subset_matches_full():
    B, H, N, d, block = 2, 2, 320, 8, 64
    Nb = N // block
    q, k, v = (_rand((B, H, N, d), s) for s in (51, 52, 53))
    kept = [[(r + t) % Nb for t in range(2)] for r in range(B * H * Nb)]
    kept = [sorted(x) for x in kept]
    row_ptr, col = _csr(kept)
    full, lf = oracle.attn_rows(q, k, v, N, block, 0.4, row_ptr, col)
    rows = [0, 7, 19, 3]
    sub, ls = oracle.attn_rows(q, k, v, N, block, 0.4, row_ptr, col, rows=rows)
    np.testing.assert_array_equal(sub, full[rows])
    np.testing.assert_array_equal(ls, lf[rows])
    dsub, _ = oracle.dense_attn_rows(q, k, v, N, block, 0.4, rows=rows)
    dfull, _ = oracle.dense_attn_rows(q, k, v, N, block, 0.4)
    np.testing.assert_array_equal(dsub, dfull[rows])
