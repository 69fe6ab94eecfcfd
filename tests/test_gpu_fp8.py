"""FP8 (e4m3 Q/K with per-block scales) variant: quantiser bytes against the oracle's, attention
against the fp64 oracle run on its own codes, dequantised (rel-L2 <= 5e-2)."""
import numpy as np
import pytest
import torch

import oracle
import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu


def _quantize(w, qd, kd):
    q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda")
    k8 = torch.zeros(kd.shape, dtype=torch.uint8, device="cuda")
    qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda")
    ks = torch.zeros_like(qs)
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    B.quantize_qk_fp8(p, qd, kd, q8, k8, qs, ks)
    torch.cuda.synchronize()
    return q8, k8, qs, ks


@pytest.mark.parametrize("name", ["even", "ragged"])
def test_quantiser_bytes_and_scales(name):
    w = shrink(WORKLOADS["large_fp8"], H=2, T=2) if name == "ragged" else shrink(WORKLOADS["medium"], H=2, T=2)
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    q8, k8, qs, ks = _quantize(w, U.dev(q), U.dev(k))
    for bits, g8, gs in ((qb, q8, qs), (kb, k8, ks)):
        codes, scales = oracle.quantize_e4m3(bits, w.N, w.block)
        np.testing.assert_array_equal(gs.cpu().numpy(), scales)
        np.testing.assert_array_equal(g8.cpu().numpy()[:, :, :w.N], codes[:, :, :w.N])
        assert (g8[:, :, w.N:] == 0).all()


@pytest.mark.parametrize("impl", ["tensor", "simt"])
def test_fp8_select_and_attention(impl):
    w = shrink(WORKLOADS["large_fp8"], H=2, T=4)          # N = 6240, ragged tail, mass rule
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    q8, k8, qs, ks = _quantize(w, qd, kd)
    qh, kh = U.oracle_fp8_inputs(w, qb, kb, q8, k8, qs, ks)
    rp, ci, sc = U.gpu_select(w, q8, k8, want_scores=True, q_scale=qs, k_scale=ks, fp8=True)
    sel, s_ref = U.oracle_select(w, qh, kh)
    assert np.abs(sc.cpu().numpy() - s_ref).max() < 2e-5
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    o, lse, st = U.gpu_attn(w, q8, k8, vd, rp, ci, simt=(impl == "simt"), q_scale=qs, k_scale=ks, fp8=True)
    assert st == 0
    rows = U.sample_rows(w.R, w.Nb, 10)
    r = U.check_attn_vs_oracle(w, qh, kh, vb, rp, ci, o, lse, rows, rel_tol=U.FP8_REL_L2, abs_tol=5e-2)
    print(f"fp8/{impl}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e}")


@pytest.mark.parametrize("impl", ["tensor", "simt", "tensor-dense"])
def test_fp8_64_token_blocks(impl):
    """e4m3 Q/K with one scale per 64-token block: the tensor-core kernel pairs blocks into 128-wide
    tiles, so the two halves of a tile (and of a tile row) carry different scales.  N = 3 * 1560 = 4680
    = 73 blocks + 8 tokens: odd block count, ragged last block."""
    w = shrink(WORKLOADS["large_fp8"], H=2, T=3, block=64, mode=0, k=9)
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    q8, k8, qs, ks = _quantize(w, qd, kd)
    qh, kh = U.oracle_fp8_inputs(w, qb, kb, q8, k8, qs, ks)
    rp, ci, _ = U.gpu_select(w, q8, k8, q_scale=qs, k_scale=ks, fp8=True)
    sel, _ = U.oracle_select(w, qh, kh)
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    dense = impl == "tensor-dense"
    o, lse, st = U.gpu_attn(w, q8, k8, vd, rp, ci, simt=(impl == "simt"), dense=dense, q_scale=qs, k_scale=ks,
                            fp8=True)
    assert st == 0
    rows = U.sample_rows(w.R, w.Nb, 6 if dense else 12)
    r = U.check_attn_vs_oracle(w, qh, kh, vb, rp, ci, o, lse, rows, dense=dense, rel_tol=U.FP8_REL_L2, abs_tol=5e-2)
    print(f"fp8 b64/{impl}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e}")


def _quantize_smooth(w, qd, kd, want_shift=True):
    q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda")
    k8 = torch.zeros(kd.shape, dtype=torch.uint8, device="cuda")
    qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda")
    ks = torch.zeros_like(qs)
    mean = torch.full((w.B, w.H, w.d), 7.0, dtype=torch.float32, device="cuda")
    shift = torch.full((w.B, w.H, w.N), 7.0, dtype=torch.float32, device="cuda") if want_shift else None
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    ws = torch.empty(B.smooth_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    B.quantize_qk_fp8_smooth_k(p, qd, kd, q8, k8, qs, ks, mean, shift, ws)
    torch.cuda.synchronize()
    return q8, k8, qs, ks, mean, shift


@pytest.mark.parametrize("block", [128, 64])
def test_smoothing_quantiser(block):
    """Mean key against the fp64 mean; K codes and scales against the oracle's quantiser run with the
    oracle's mean; Q untouched by the smoothing; lse shift against its definition."""
    w = shrink(WORKLOADS["large_fp8"], H=2, T=2, block=block)         # N = 3120, ragged
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    qd, kd = U.dev(q), U.dev(k)
    q8, k8, qs, ks, mean, shift = _quantize_smooth(w, qd, kd)
    m = mean.cpu().numpy()
    m_ref = oracle.k_mean(kb, w.N)
    assert np.abs(m - m_ref).max() <= 1e-5 * max(1.0, np.abs(m_ref).max())
    # the oracle quantises with its own mean (rounded to fp32, the precision the subtraction is defined in); the
    # GPU's mean differs from it in the last bits, which can move a value across a rounding boundary of the
    # cast once in about a million elements: scales to 1e-6, codes equal but for a handful one step apart
    codes, scales = oracle.quantize_e4m3(kb, w.N, w.block, sub=m_ref.astype(np.float32))
    np.testing.assert_allclose(ks.cpu().numpy(), scales, rtol=2e-6)
    g8 = k8.cpu().numpy()[:, :, :w.N]
    differ = g8 != codes[:, :, :w.N]
    assert differ.mean() < 1e-4, differ.mean()
    dq_g = oracle.dequantize_e4m3(k8.cpu().numpy(), ks.cpu().numpy(), w.N, w.block)[:, :, :w.N]
    dq_o = oracle.dequantize_e4m3(codes, scales, w.N, w.block)[:, :, :w.N]
    step = np.repeat(scales.astype(np.float64), w.block, axis=-1)[:, :, :w.N, None] * 32.0     # the widest e4m3 step (at 256..448) times the scale
    assert (np.abs(dq_g - dq_o) <= step).all()
    assert (k8[:, :, w.N:] == 0).all()
    qc, qsc = oracle.quantize_e4m3(qb, w.N, w.block)
    np.testing.assert_array_equal(qs.cpu().numpy(), qsc)
    np.testing.assert_array_equal(q8.cpu().numpy()[:, :, :w.N], qc[:, :, :w.N])
    s_ref = oracle.lse_shift(qb, m_ref, w.N, w.scale)
    assert np.abs(shift.cpu().numpy() - s_ref).max() <= 1e-4 * max(1.0, np.abs(s_ref).max())
    # the shift is optional
    _quantize_smooth(w, qd, kd, want_shift=False)


def test_smoothed_fp8_attention_is_closer_to_bf16_attention():
    """Routing + attention on the smoothed codes: parity against the oracle on the dequantised
    inputs (same tolerances as the plain FP8 variant), lse + shift against the oracle's lse of the
    un-smoothed problem, and -- what the step is for -- a smaller distance to the attention of the
    original bf16 Q, K than the plain FP8 variant has, on inputs whose keys share an offset."""
    w = shrink(WORKLOADS["large_fp8"], H=2, T=4)
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    g = torch.Generator().manual_seed(11)
    k = (k.float() + 3.0 * torch.randn(w.B, w.H, 1, w.d, generator=g)).bfloat16()   # one offset per head, 3x the noise
    k[:, :, w.N:] = 0
    kb = k.view(torch.int16).numpy().view(np.uint16)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    # Q, K of this test are the oracle's smoothed codes and scales, given to both sides (the GPU's smoothing
    # quantiser has its own test above); the lse shift is the GPU's
    _, _, _, _, mean, shift = _quantize_smooth(w, qd, kd)
    m32 = oracle.k_mean(kb, w.N).astype(np.float32)
    cq, sq_ = oracle.quantize_e4m3(qb, w.N, w.block)
    ck, sk_ = oracle.quantize_e4m3(kb, w.N, w.block, sub=m32)
    q8, k8 = torch.from_numpy(cq).cuda(), torch.from_numpy(ck).cuda()
    qs, ks = torch.from_numpy(sq_).cuda(), torch.from_numpy(sk_).cuda()
    qh = oracle.dequantize_e4m3(cq, sq_, w.N, w.block)
    kh = oracle.dequantize_e4m3(ck, sk_, w.N, w.block)
    rp, ci, _ = U.gpu_select(w, q8, k8, q_scale=qs, k_scale=ks, fp8=True)
    sel, _ = U.oracle_select(w, qh, kh)
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    o, lse, st = U.gpu_attn(w, q8, k8, vd, rp, ci, q_scale=qs, k_scale=ks, fp8=True)
    assert st == 0
    rows = U.sample_rows(w.R, w.Nb, 10)
    U.check_attn_vs_oracle(w, qh, kh, vb, rp, ci, o, lse, rows, rel_tol=U.FP8_REL_L2, abs_tol=5e-2)
    rpn, cin = rp.cpu().numpy(), ci.cpu().numpy()
    # distance to the attention of the original bf16 inputs over the same block lists
    # (lse: the smoothed problem's plus the shift, which is taken from the bf16 q, estimates the original's)
    o_true, l_true = oracle.attn_rows(qb, kb, vb, w.N, w.block, w.scale, rpn, cin, rows=rows)
    _, e_smooth, l_smooth = U.attn_errors(o, lse + shift, o_true, l_true, rows, w.N, w.block, w.H)
    p8, pk8, pqs, pks = _quantize(w, qd, kd)
    o_plain, lse_plain, st = U.gpu_attn(w, p8, pk8, vd, rp, ci, q_scale=pqs, k_scale=pks, fp8=True)
    _, e_plain, l_plain = U.attn_errors(o_plain, lse_plain, o_true, l_true, rows, w.N, w.block, w.H)
    print(f"to bf16 attention: rel-L2 plain fp8 {e_plain:.3e}, smoothed {e_smooth:.3e}; "
          f"max lse error plain {l_plain:.3e}, smoothed {l_smooth:.3e}")
    assert e_smooth < e_plain and l_smooth < l_plain


def test_quantiser_every_bf16_value_under_many_scales():
    """The cast divides by the block scale with a short exact-division sequence: every finite bf16 value
    (both zeros, subnormals) not above the block's absmax, under absmax values spread over the exponent
    range (among them significands of all ones and the extremes that take the general division), bit for
    bit against the oracle."""
    pat = np.arange(1 << 16, dtype=np.uint32).astype(np.uint16)
    val = torch.from_numpy(pat.view(np.int16)).view(torch.bfloat16).float().numpy()
    fin = np.isfinite(val)
    rng = np.random.default_rng(5)
    amax_bits = [0x3F80, 0x3FFF, 0x7F7F, 0x0080, 0x0001, 0x5F7F, 0x1F01] + \
                [int(e) << 7 | int(m) for e, m in zip(rng.integers(60, 200, 9), rng.integers(0, 128, 9))]
    blocks = []
    for ab in amax_bits:
        a = val[ab]
        mine = pat[fin & (np.abs(val) <= a)]
        for lo in range(0, mine.size, 16383):
            blk = np.zeros(16384, np.uint16)
            chunk = mine[lo:lo + 16383]
            blk[:chunk.size] = chunk
            blk[-1] = ab                                              # the block's absmax is always present
            blocks.append(blk.reshape(128, 128))
    x = np.stack(blocks).reshape(1, 1, -1, 128)
    N = x.shape[2]
    xt = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda()
    w = shrink(WORKLOADS["large_fp8"], H=1, T=1)
    q8 = torch.zeros(xt.shape, dtype=torch.uint8, device="cuda"); k8 = torch.zeros_like(q8)
    qs = torch.zeros(1, 1, N // 128, dtype=torch.float32, device="cuda"); ks = torch.zeros_like(qs)
    p = B.make_problem(xt, xt, None, None, N, 128)
    B.quantize_qk_fp8(p, xt, xt, q8, k8, qs, ks)
    torch.cuda.synchronize()
    codes, scales = oracle.quantize_e4m3(x, N, 128)
    np.testing.assert_array_equal(qs.cpu().numpy(), scales)
    np.testing.assert_array_equal(q8.cpu().numpy(), codes)
    np.testing.assert_array_equal(k8.cpu().numpy(), codes)


@pytest.mark.parametrize("block", [128, 64])
def test_fp8_d64(block):
    """e4m3 Q/K with d = 64 (the tensor-core kernel computes it as d = 128 with a zero upper half)."""
    w = shrink(WORKLOADS["large_fp8"], H=2, T=3, d=64, block=block, mode=0, k=7)
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    q8, k8, qs, ks = _quantize(w, qd, kd)
    qh, kh = U.oracle_fp8_inputs(w, qb, kb, q8, k8, qs, ks)
    rp, ci, _ = U.gpu_select(w, q8, k8, q_scale=qs, k_scale=ks, fp8=True)
    o, lse, st = U.gpu_attn(w, q8, k8, vd, rp, ci, q_scale=qs, k_scale=ks, fp8=True)
    assert st == 0
    rows = U.sample_rows(w.R, w.Nb, 12)
    r = U.check_attn_vs_oracle(w, qh, kh, vb, rp, ci, o, lse, rows, rel_tol=U.FP8_REL_L2, abs_tol=5e-2)
    o2, lse2, st2 = U.gpu_attn(w, q8, k8, vd, rp, ci, simt=True, q_scale=qs, k_scale=ks, fp8=True)
    print(f"fp8 d64 block {block}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e}; vs simt max diff {(o.float() - o2.float()).abs().max().item():.2e}")


def test_fp8_two_step_form_matches_the_one_call_form():
    w = shrink(WORKLOADS["large_fp8"], H=2, T=4)
    (q, k, v), _ = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    q8, k8, qs, ks = _quantize(w, qd, kd)
    rp, ci, _ = U.gpu_select(w, q8, k8, q_scale=qs, k_scale=ks, fp8=True)
    o1, l1, st = U.gpu_attn(w, q8, k8, vd, rp, ci, q_scale=qs, k_scale=ks, fp8=True)
    o2 = torch.full_like(o1, 3.0); l2 = torch.full_like(l1, 3.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = B.make_problem(q8, k8, vd, o2, w.N, w.block, 0.0, True)
    ws = torch.full((B.attn_workspace_bytes(p),), 0xFF, dtype=torch.uint8, device="cuda")
    B.attn_prepare_v(p, vd, ws)
    for _ in range(2):                                    # the prepared workspace serves repeated calls
        o2.fill_(3.0); l2.fill_(3.0)
        B.block_sparse_attn_fwd_prepared(p, q8, k8, rp, ci, o2, l2, status, workspace=ws, q_scale=qs, k_scale=ks)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(o2[:, :, :w.N], o1[:, :, :w.N]) and torch.equal(l2, l1)
