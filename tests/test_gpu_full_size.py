"""Full-size configurations in the launch configuration the bench times: selection parity on
every row; attention parity against the oracle on a per-head sample of query blocks (for EVERY (b, h):
block 0, the ragged last block and 8 seeded random ones, which the oracle computes one by one); and every
element of O and LSE against the CUDA-core kernel of the same contract (a supplement that reaches the rows
the oracle sample leaves out -- the oracle stays the judge)."""
import numpy as np
import pytest
import torch

import oracle
import _util as U
from paper_2606_23743_b200.workloads import WORKLOADS

pytestmark = pytest.mark.gpu


def check_against_twin(w, qd, kd, vd, rp, ci, o, lse, q_scale=None, k_scale=None, fp8=False):
    """Every valid element of O and LSE of the tensor-core kernel against the CUDA-core kernel run on the same
    CSR (fp32 arithmetic, one thread per query row: a different program, the same contract)."""
    o2, lse2, st2 = U.gpu_attn(w, qd, kd, vd, rp, ci, simt=True, q_scale=q_scale, k_scale=k_scale, fp8=fp8)
    assert st2 == 0
    a, b = o[:, :, :w.N].float(), o2[:, :, :w.N].float()
    diff = (a - b).abs()
    # both sides round to bf16 (half a unit each) around results that differ by the bf16 rounding of P
    excess = diff - torch.clamp(b.abs() * 2.0 ** -7, min=(5e-2 if fp8 else U.BF16_MAX_ABS))   # (large outputs: one bf16 unit)
    assert float(excess.max()) <= 0.0, float(excess.max())
    worst = float(diff.max())
    rel = float(torch.linalg.vector_norm(a - b) / torch.linalg.vector_norm(b))
    lerr = float((lse - lse2).abs().max())
    # per query block: no block of rows may stand out (a row handed out twice, a skipped tile)
    per_block = diff.reshape(w.B * w.H, -1).amax(dim=1)
    assert rel <= (2e-2 if fp8 else U.BF16_REL_L2) and lerr <= 2e-3, (worst, rel, lerr)
    assert torch.isfinite(a).all() and torch.isfinite(lse).all()
    return worst, rel, lerr, float(per_block.max())


@pytest.mark.parametrize("name", ["medium", "large", "xl", "large_b64"])
def test_full_size_select_then_attend(name):
    w = WORKLOADS[name]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, _ = U.gpu_select(w, qd, kd)
    sel, _ = U.oracle_select(w, qb, kb)
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    print(f"{name}: rows {w.R} nnz {ci.numel()} differing {n_diff} near-tie rows {n_near}")
    assert n_diff <= n_near
    o, lse, st = U.gpu_attn(w, qd, kd, vd, rp, ci)
    assert st == 0
    rows = U.sample_rows_per_head(w.B * w.H, w.Nb, 8, seed=w.cfg)
    r = U.check_attn_vs_oracle(w, qb, kb, vb, rp, ci, o, lse, rows)
    print(f"{name}: oracle sample {len(rows)} of {w.R} query blocks (10 per head): max_abs {r[0]:.2e} rel_l2 {r[1]:.2e} lse {r[2]:.2e}")
    t = check_against_twin(w, qd, kd, vd, rp, ci, o, lse)
    print(f"{name}: every element vs the CUDA-core kernel: max_abs {t[0]:.2e} rel_l2 {t[1]:.2e} lse {t[2]:.2e}")
    # properties that hold at any size: finite outputs inside V's range, rows never written past N
    of = o[:, :, :w.N].float()
    assert torch.isfinite(of).all()
    vmax = vd[:, :, :w.N].float().abs().amax()
    assert of.abs().amax() <= vmax * 1.01
    if w.n_alloc > w.N:
        assert (o[:, :, w.N:] == 7.0).all()
    if name == "large":
        # the launch configuration bench.py times: V prepared on a second stream, then the kernel alone
        from paper_2606_23743_b200 import binding as B
        o2 = torch.full_like(o, 7.0); lse2 = torch.full_like(lse, 7.0)
        st2 = torch.zeros(1, dtype=torch.int32, device="cuda")
        p = B.make_problem(qd, kd, vd, o2, w.N, w.block)
        aws = torch.full((B.attn_workspace_bytes(p),), 0xFF, dtype=torch.uint8, device="cuda")
        side, ready = torch.cuda.Stream(), torch.cuda.Event()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            B.attn_prepare_v(p, vd, aws)
            ready.record()
        torch.cuda.current_stream().wait_event(ready)
        B.block_sparse_attn_fwd_prepared(p, qd, kd, rp, ci, o2, lse2, st2, workspace=aws)
        torch.cuda.synchronize()
        assert int(st2.item()) == 0 and torch.equal(o2, o) and torch.equal(lse2, lse)
    if name == "medium":
        od, lsd, _ = U.gpu_attn(w, qd, kd, vd, None, None, dense=True)
        U.check_attn_vs_oracle(w, qb, kb, vb, None, None, od, lsd, rows[:4], dense=True)


def test_full_size_fp8():
    from paper_2606_23743_b200 import binding as B
    w = WORKLOADS["large_fp8"]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda"); k8 = torch.zeros_like(q8)
    qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda"); ks = torch.zeros_like(qs)
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    B.quantize_qk_fp8(p, qd, kd, q8, k8, qs, ks)
    torch.cuda.synchronize()
    # the quantiser at full size, bit for bit
    for bits, g8, gs in ((qb, q8, qs), (kb, k8, ks)):
        codes, scales = oracle.quantize_e4m3(bits, w.N, w.block)
        np.testing.assert_array_equal(gs.cpu().numpy(), scales)
        assert np.array_equal(g8.cpu().numpy()[:, :, :w.N], codes[:, :, :w.N])
    qh, kh = U.oracle_fp8_inputs(w, qb, kb, q8, k8, qs, ks)
    rp, ci, _ = U.gpu_select(w, q8, k8, q_scale=qs, k_scale=ks, fp8=True)
    sel, _ = U.oracle_select(w, qh, kh)
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    o, lse, st = U.gpu_attn(w, q8, k8, vd, rp, ci, q_scale=qs, k_scale=ks, fp8=True)
    assert st == 0
    rows = U.sample_rows_per_head(w.B * w.H, w.Nb, 8, seed=5)
    r = U.check_attn_vs_oracle(w, qh, kh, vb, rp, ci, o, lse, rows, rel_tol=U.FP8_REL_L2, abs_tol=5e-2)
    print(f"large_fp8: differing {n_diff} near {n_near}; oracle sample {len(rows)} of {w.R}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e}")
    t = check_against_twin(w, q8, k8, vd, rp, ci, o, lse, q_scale=qs, k_scale=ks, fp8=True)
    print(f"large_fp8: every element vs the CUDA-core kernel: max_abs {t[0]:.2e} rel_l2 {t[1]:.2e} lse {t[2]:.2e}")


def test_full_size_prologue():
    """The fused QK-norm + RoPE prologue in the launch configuration `bench.py --prologue` times
    (cfg 5 shape: bf16 write-back, block means and e4m3 codes in one launch): three sampled heads against
    the oracle, then routing from its means against routing that pools the written Q, K itself."""
    from paper_2606_23743_b200 import binding as B
    from paper_2606_23743_b200.workloads import bf16_bits, make_prologue_inputs
    w = WORKLOADS["large_fp8"]
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    qd, kd = U.dev(q), U.dev(k)
    gq, gk, cos, sin = make_prologue_inputs(w)
    qo, ko = torch.full_like(qd, 7.0), torch.full_like(kd, 7.0)
    qm = torch.zeros(w.B, w.H, w.Nb, w.d, dtype=torch.float32, device="cuda"); km = torch.zeros_like(qm)
    q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda"); k8 = torch.zeros_like(q8)
    qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda"); ks = torch.zeros_like(qs)
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    B.qk_norm_rope_pool(p, qd, kd, gq.cuda(), gk.cuda(), cos.cuda(), sin.cuda(), 1e-6, qo, ko, qm, km, q8, k8, qs, ks)
    torch.cuda.synchronize()
    for h in (0, 11, w.H - 1):
        for bits, g, out, mean, c8, sc in ((qb, gq, qo, qm, q8, qs), (kb, gk, ko, km, k8, ks)):
            ref = oracle.qk_norm_rope(bits[:, h:h + 1], g.numpy(), cos.numpy(), sin.numpy(), w.N, 1e-6)[:, :, :w.N]
            got = out[:, h:h + 1, :w.N].float().cpu().numpy().astype(np.float64)
            assert (np.abs(got - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-5).all()
            assert (got == torch.from_numpy(ref).to(torch.bfloat16).float().numpy()).mean() > 0.999
            ob = bf16_bits(out[:, h:h + 1].cpu())
            np.testing.assert_allclose(mean[:, h:h + 1].cpu().numpy(), oracle.pool(ob, w.N, w.block), rtol=2e-6, atol=2e-7)
            codes, scales = oracle.quantize_e4m3(ob, w.N, w.block)
            np.testing.assert_array_equal(sc[:, h:h + 1].cpu().numpy(), scales)
            assert np.array_equal(c8[:, h:h + 1, :w.N].cpu().numpy(), codes[:, :, :w.N])
    assert (qo[:, :, w.N:] == 7.0).all() and (ko[:, :, w.N:] == 7.0).all()
    s = B.make_select(w.mode, w.k, w.tau)
    pb = B.make_problem(qo, ko, None, None, w.N, w.block)
    rp = torch.zeros(w.R + 1, dtype=torch.int32, device="cuda")
    ci = torch.zeros(B.select_max_nnz(pb, s), dtype=torch.int32, device="cuda")
    ws = torch.empty(B.select_workspace_bytes(pb, s), dtype=torch.uint8, device="cuda")
    B.block_select_pooled(pb, s, qm, km, rp, ci, ws)
    torch.cuda.synchronize()
    rp2, ci2, _ = U.gpu_select(w, qo, ko)          # (bf16 routing: gpu_select takes the dtype from its fp8 argument)
    assert torch.equal(rp, rp2) and torch.equal(ci[: int(rp[-1])], ci2)


@pytest.mark.parametrize("name,order", [("large", 0), ("large_b64", 0), ("large", 1), ("large_b64", 1)])
def test_full_size_remainder(name, order):
    """Piecewise attention with the remainder at full size in the launch configuration `bench.py --remainder
    [--remainder-order 1]` times: per head, block 0, the ragged last block and 3 random ones against the oracle
    (order 1: four heads -- the oracle's d x d block statistics are numpy)."""
    from test_gpu_remainder import check_vs_oracle, gpu_remainder
    w = WORKLOADS[name]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, scores = U.gpu_select(w, qd, kd, want_scores=order == 1)
    o, lse, st = gpu_remainder(w, qd, kd, vd, rp, ci, order, scores=scores)
    assert st == 0
    if order == 0:
        rows = U.sample_rows_per_head(w.B * w.H, w.Nb, 3, seed=w.cfg)
        r = check_vs_oracle(w, qb, kb, vb, rp, ci, o, lse, rows)
    else:
        from paper_2606_23743_b200.workloads import shrink
        r = (0.0, 0.0, 0.0)
        rows = []
        for h in (0, 9, 17, w.H - 1):
            w1 = shrink(w, H=1)
            rp_h = (rp[h * w.Nb:(h + 1) * w.Nb + 1] - rp[h * w.Nb]).cpu()
            ci_h = ci[int(rp[h * w.Nb]):int(rp[(h + 1) * w.Nb])].cpu()
            rows_h = U.sample_rows_per_head(1, w.Nb, 3, seed=h)
            rh = check_vs_oracle(w1, qb[:, h:h + 1], kb[:, h:h + 1], vb[:, h:h + 1], rp_h, ci_h, o[:, h:h + 1], lse[:, h:h + 1],
                                 rows_h, 1)
            r = tuple(max(a, b) for a, b in zip(r, rh)); rows += rows_h
    print(f"{name} + remainder order {order}: oracle sample {len(rows)} of {w.R} query blocks: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e} lse {r[2]:.2e}")
    assert torch.isfinite(o[:, :, :w.N].float()).all() and torch.isfinite(lse).all()
    if w.n_alloc > w.N:
        assert (o[:, :, w.N:] == 7.0).all()
