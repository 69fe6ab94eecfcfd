"""Pins for the oracle's approximate remainder (the paper's "first-order Taylor" compensation of dropped
blocks, as this build reads it): none of them re-types the block-statistics form the oracle uses."""
import numpy as np
import pytest

import oracle


def _csr(kept):
    row_ptr = np.zeros(len(kept) + 1, np.int32)
    row_ptr[1:] = np.cumsum([len(x) for x in kept])
    col = np.concatenate([np.asarray(x, np.int32) for x in kept]) if row_ptr[-1] else np.zeros(0, np.int32)
    return row_ptr, col


def _case(N=200, block=32, d=8, B=1, H=2, seed=0, keep=2):
    rng = np.random.default_rng(seed)
    Nb = -(-N // block)
    q, k, v = (rng.standard_normal((B, H, Nb * block, d)) for _ in range(3))
    q[:, :, N:] = 7.0; k[:, :, N:] = -5.0; v[:, :, N:] = 9.0          # the absent tail must not matter
    kept = [sorted(rng.choice(Nb, size=keep, replace=False).tolist()) for _ in range(B * H * Nb)]
    return q, k, v, kept, Nb


def _dense(q, k, v, N, scale):
    S = scale * np.einsum("bhid,bhjd->bhij", q[:, :, :N], k[:, :, :N])
    m = S.max(-1, keepdims=True)
    P = np.exp(S - m)
    return np.einsum("bhij,bhjd->bhid", P, v[:, :, :N]) / P.sum(-1, keepdims=True), (m + np.log(P.sum(-1, keepdims=True)))[..., 0]


def _unblock(o, B, H, N, block):
    Nb = -(-N // block)
    return o.reshape(B, H, Nb * block, *o.shape[2:])[:, :, :N]


def _per_key_reference(q, k, v, N, block, scale, kept, order, weight):
    """The same expansion written per KEY instead of per block statistic: every dropped key j of block J gets
    the weight exp(a_iJ) + w1 * scale <q_i, k_j - kbar_J>, w1 = exp(a_iJ) or exp(sbar_IJ); no C_J is formed."""
    B, H, _, d = q.shape
    Nb = -(-N // block)
    out = np.zeros((B, H, N, d)); lse = np.zeros((B, H, N))
    blk = np.arange(N) // block
    for b in range(B):
        for h in range(H):
            K, V, Q = k[b, h, :N], v[b, h, :N], q[b, h, :N]
            kbar = np.stack([K[blk == J].mean(0) for J in range(Nb)])
            qbar = np.stack([Q[blk == J].mean(0) for J in range(Nb)])
            for i in range(N):
                I = i // block
                ks = set(kept[(b * H + h) * Nb + I])
                num, den = np.zeros(d), 0.0
                for j in range(N):
                    J = j // block
                    if J in ks:
                        wgt = np.exp(scale * Q[i] @ K[j])
                    else:
                        a = np.exp(scale * Q[i] @ kbar[J])
                        wgt = a
                        if order == 1:
                            w1 = a if weight == "query" else np.exp(scale * qbar[I] @ kbar[J])
                            wgt = a + w1 * scale * (Q[i] @ (K[j] - kbar[J]))
                    num += wgt * V[j]; den += wgt
                out[b, h, i] = num / den; lse[b, h, i] = np.log(den)
    return out, lse


@pytest.mark.parametrize("order,weight", [(0, "block"), (1, "block"), (1, "query")])
def test_per_key_form_of_the_same_expansion(order, weight):
    N, block = 100, 16
    q, k, v, kept, Nb = _case(N=N, block=block, d=6, H=1, seed=3, keep=2)
    kept[3] = []                                      # a query block that keeps nothing: all remainder
    rp, ci = _csr(kept)
    scale = 0.3
    o, lse = oracle.attn_remainder_rows(q, k, v, N, block, scale, rp, ci, range(Nb), order=order, order1_weight=weight)
    ref_o, ref_l = _per_key_reference(q, k, v, N, block, scale, kept, order, weight)
    np.testing.assert_allclose(_unblock(o, 1, 1, N, block), ref_o, rtol=1e-10, atol=1e-12)
    # (the first-order terms of the denominator cancel inside every block, so the per-key weights sum to Z)
    np.testing.assert_allclose(_unblock(lse, 1, 1, N, block), ref_l, rtol=1e-10, atol=1e-12)


def test_keep_all_has_no_remainder_and_is_dense():
    """Nothing dropped: the exact result comes back bit for bit (no merge arithmetic touches it), and it is
    dense attention (the oracle's dense routine normalises in another order: equal to rounding)."""
    N, block = 200, 32
    q, k, v, _, Nb = _case(N=N, block=block)
    rp, ci = _csr([list(range(Nb))] * (2 * Nb))
    o, lse = oracle.attn_remainder_rows(q, k, v, N, block, 0.35, rp, ci, range(2 * Nb))
    o_e, lse_e = oracle.attn_rows(q, k, v, N, block, 0.35, rp, ci)
    assert np.array_equal(o, o_e, equal_nan=True) and np.array_equal(lse, lse_e, equal_nan=True)
    o_d, lse_d = _dense(q, k, v, N, 0.35)
    np.testing.assert_allclose(_unblock(o, 1, 2, N, block), o_d, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(_unblock(lse, 1, 2, N, block), lse_d, rtol=1e-13)


@pytest.mark.parametrize("order", [0, 1])
def test_identical_keys_inside_dropped_blocks_make_the_expansion_exact(order):
    N, block = 176, 16
    q, k, v, kept, Nb = _case(N=N, block=block, d=8, H=2, seed=5, keep=3)
    for J in range(Nb):                               # every block: one key repeated (values stay distinct)
        k[:, :, J * block:(J + 1) * block] = k[:, :, J * block:J * block + 1]
    rp, ci = _csr(kept)
    o, lse = oracle.attn_remainder_rows(q, k, v, N, block, 0.4, rp, ci, range(2 * Nb), order=order)
    o_d, lse_d = _dense(q, k, v, N, 0.4)
    np.testing.assert_allclose(_unblock(o, 1, 2, N, block), o_d, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(_unblock(lse, 1, 2, N, block), lse_d, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("order", [0, 1])
def test_weights_sum_to_one(order):
    """Constant V: whatever the weights are, they must sum to one (the first-order terms cancel per block)."""
    N, block = 150, 32
    q, k, v, kept, Nb = _case(N=N, block=block, seed=7)
    c = np.array([1.5, -2.0, 0.25, 3.0, 0.0, -1.0, 2.0, 0.5])
    v[:] = c
    rp, ci = _csr(kept)
    o, _ = oracle.attn_remainder_rows(q, k, v, N, block, 0.3, rp, ci, range(2 * Nb), order=order)
    got = _unblock(o, 1, 2, N, block)
    np.testing.assert_allclose(got, np.broadcast_to(c, got.shape), rtol=1e-12, atol=1e-12)


def test_lse_is_the_logaddexp_of_the_two_parts_and_merge_matches_direct_sums():
    N, block = 200, 32
    q, k, v, kept, Nb = _case(N=N, block=block, seed=11)
    rp, ci = _csr(kept)
    rows = list(range(2 * Nb))
    o, lse = oracle.attn_remainder_rows(q, k, v, N, block, 0.3, rp, ci, rows)
    o_e, lse_e = oracle.attn_rows(q, k, v, N, block, 0.3, rp, ci, rows=rows)
    o_r, lnz_r = oracle.remainder_rows(q, k, v, N, block, 0.3, rp, ci, rows)
    ok = ~np.isnan(lse)
    np.testing.assert_allclose(lse[ok], np.logaddexp(lse_e[ok], lnz_r[ok]), rtol=1e-13)
    num = np.exp(lse_e)[..., None] * o_e + np.exp(lnz_r)[..., None] * o_r
    np.testing.assert_allclose(o[ok], (num / (np.exp(lse_e) + np.exp(lnz_r))[..., None])[ok], rtol=1e-11, atol=1e-13)


def test_error_against_dense_is_of_second_order():
    """Keys and queries = block means + eps * noise: halving eps must quarter the first-order result's
    distance to dense attention (the dropped terms are quadratic in the deviations); order 0 is
    first-order accurate only in its numerator, so it merely halves."""
    N, block, d, H = 128, 16, 8, 1
    Nb = N // block
    rng = np.random.default_rng(13)
    qc, kc = rng.standard_normal((Nb, d)), rng.standard_normal((Nb, d))
    nq, nk = rng.standard_normal((N, d)), rng.standard_normal((N, d))
    v = rng.standard_normal((1, H, N, d))
    kept = [[I] for I in range(Nb)]
    rp, ci = _csr(kept)
    errs = {0: [], 1: []}
    for eps in (0.08, 0.04, 0.02):
        q = (np.repeat(qc, block, 0) + eps * nq)[None, None]
        k = (np.repeat(kc, block, 0) + eps * nk)[None, None]
        o_d, _ = _dense(q, k, v, N, 0.5)
        for order in (0, 1):
            o, _ = oracle.attn_remainder_rows(q, k, v, N, block, 0.5, rp, ci, range(Nb), order=order)
            errs[order].append(np.abs(_unblock(o, 1, 1, N, block) - o_d).max())
    r1 = [errs[1][i] / errs[1][i + 1] for i in range(2)]
    r0 = [errs[0][i] / errs[0][i + 1] for i in range(2)]
    assert all(3.5 < r < 4.5 for r in r1), r1
    assert all(1.7 < r < 2.4 for r in r0), r0
    assert errs[1][-1] < errs[0][-1] / 10


def test_bf16_statistics_are_the_rounded_exact_ones():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -9, -0.3, 3.0e38, 1e-40])
    import torch
    ref = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    from oracle.remainder import _round_bf16
    np.testing.assert_array_equal(_round_bf16(x), ref)
    N, block = 96, 32
    q, k, v, kept, Nb = _case(N=N, block=block, seed=17)
    rp, ci = _csr(kept)
    a, _ = oracle.attn_remainder_rows(q, k, v, N, block, 0.3, rp, ci, range(2 * Nb), stats="f64")
    b, _ = oracle.attn_remainder_rows(q, k, v, N, block, 0.3, rp, ci, range(2 * Nb), stats="bf16")
    ok = ~np.isnan(a)
    assert 0 < np.abs(a[ok] - b[ok]).max() < 2e-2
