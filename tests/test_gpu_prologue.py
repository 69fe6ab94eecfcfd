"""Fused QK-norm + RoPE (+ block means, + e4m3 codes) prologue and routing from its block means."""
import numpy as np
import pytest
import torch

import oracle
import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, bf16_bits, make_prologue_inputs, shrink

pytestmark = pytest.mark.gpu
EPS = 1e-6


def _run(w, q, k, fp8=False, in_place=False, means=True):
    gq, gk, cos, sin = make_prologue_inputs(w)
    qd, kd = U.dev(q), U.dev(k)
    qo = qd if in_place else torch.full_like(qd, 7.0)
    ko = kd if in_place else torch.full_like(kd, 7.0)
    qm = torch.full((w.B, w.H, w.Nb, w.d), 7.0, dtype=torch.float32, device="cuda") if means else None
    km = torch.full_like(qm, 7.0) if means else None
    q8 = k8 = qs = ks = None
    if fp8:
        q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda"); k8 = torch.zeros_like(q8)
        qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda"); ks = torch.zeros_like(qs)
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    B.qk_norm_rope_pool(p, qd, kd, gq.cuda(), gk.cuda(), cos.cuda(), sin.cuda(), EPS, qo, ko, qm, km, q8, k8, qs, ks)
    torch.cuda.synchronize()
    return (gq, gk, cos, sin), qo, ko, qm, km, q8, k8, qs, ks


def _check_rounded(out, ref, N):
    """out: bf16 device tensor; ref: fp64 oracle values (O(1) here).  Within one bf16 unit of the exact
    value everywhere (the kernel computes in fp32), and the correctly rounded value almost everywhere."""
    got = out.float().cpu().numpy().astype(np.float64)[:, :, :N]
    ref = ref[:, :, :N]
    # (2^-7 relative: one bf16 unit; the absolute term covers fp32 cancellation in a rotated pair near zero)
    assert (np.abs(got - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-5).all()
    exact = torch.from_numpy(ref).to(torch.bfloat16).float().numpy()
    frac = (got == exact).mean()
    assert frac > 0.999, frac
    return frac


@pytest.mark.parametrize("name,block,in_place", [("medium", 128, False), ("large", 128, True), ("large", 64, False),
                                                 ("tiny", 64, False)])
def test_prologue_outputs(name, block, in_place):
    w = shrink(WORKLOADS[name], H=2, T=2, block=block) if name != "tiny" else WORKLOADS["tiny"]
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    (gq, gk, cos, sin), qo, ko, qm, km, *_ = _run(w, q, k, in_place=in_place)
    for bits, g, out, mean in ((qb, gq, qo, qm), (kb, gk, ko, km)):
        ref = oracle.qk_norm_rope(bits, g.numpy(), cos.numpy(), sin.numpy(), w.N, EPS)
        _check_rounded(out, ref, w.N)
        if not in_place:
            assert (out[:, :, w.N:] == 7.0).all()                     # rows that do not exist are not written
        # the means against the oracle's own chain (its Q', K' rounded to bf16, then pooled): the few elements
        # the two sides round differently move a block mean by a fraction of a bf16 unit at most ...
        ref_bits = bf16_bits(torch.from_numpy(ref).to(torch.bfloat16))
        np.testing.assert_allclose(mean.cpu().numpy(), oracle.pool(ref_bits, w.N, w.block), rtol=0, atol=2e-4)
        # ... and, as a property of the kernel's outputs among themselves, they are the means of the values written
        m_ref = oracle.pool(bf16_bits(out.cpu()), w.N, w.block)
        np.testing.assert_allclose(mean.cpu().numpy(), m_ref, rtol=2e-6, atol=2e-7)


def test_prologue_codes_match_the_quantiser():
    """A property of the kernel's outputs among themselves: the codes and scales are what the (oracle's)
    quantiser makes of the bf16 values the same launch wrote."""
    w = shrink(WORKLOADS["large_fp8"], H=2, T=2)
    (q, k, _), _ = U.host_inputs(w)
    _, qo, ko, qm, km, q8, k8, qs, ks = _run(w, q, k, fp8=True, means=False)
    for out, g8, gs in ((qo, q8, qs), (ko, k8, ks)):
        codes, scales = oracle.quantize_e4m3(bf16_bits(out.cpu()), w.N, w.block)
        np.testing.assert_array_equal(gs.cpu().numpy(), scales)
        np.testing.assert_array_equal(g8.cpu().numpy()[:, :, :w.N], codes[:, :, :w.N])
        assert (g8[:, :, w.N:] == 0).all()


@pytest.mark.parametrize("name", ["large", "medium"])
def test_routing_from_the_prologue_means_and_attention(name):
    """prologue -> routing from its means -> attention, against the oracle run on the Q, K the prologue wrote."""
    w = shrink(WORKLOADS[name], H=2, T=4)
    (q, k, v), (_, _, vb) = U.host_inputs(w)
    _, qo, ko, qm, km, *_ = _run(w, q, k)
    p = B.make_problem(qo, ko, None, None, w.N, w.block)
    s = B.make_select(w.mode, w.k, w.tau, w.win_t, w.win_s, w.blocks_per_frame if w.win_t >= 0 else 0)
    rp = torch.zeros(w.R + 1, dtype=torch.int32, device="cuda")
    ci = torch.zeros(B.select_max_nnz(p, s), dtype=torch.int32, device="cuda")
    sc = torch.zeros(w.B, w.H, w.Nb, w.Nb, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.select_workspace_bytes(p, s), dtype=torch.uint8, device="cuda")
    B.block_select_pooled(p, s, qm, km, rp, ci, ws, block_scores=sc)
    torch.cuda.synchronize()
    ci = ci[: int(rp[-1].item())]
    qob, kob = bf16_bits(qo.cpu()), bf16_bits(ko.cpu())
    sel, s_ref = U.oracle_select(w, qob, kob)
    assert np.abs(sc.cpu().numpy() - s_ref).max() < 2e-5 * max(1.0, np.abs(s_ref).max())
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    # the same lists as the routing that pools by itself
    rp2, ci2, _ = U.gpu_select(w, qo, ko)
    assert torch.equal(rp, rp2) and torch.equal(ci, ci2)
    o, lse, st = U.gpu_attn(w, qo, ko, U.dev(v), rp, ci)
    assert st == 0
    U.check_attn_vs_oracle(w, qob, kob, vb, rp, ci, o, lse, U.sample_rows(w.R, w.Nb, 8))
