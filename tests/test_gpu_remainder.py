"""Piecewise attention with the approximate remainder (orders 0 and 1) through the C ABI against the oracle's
remainder formula with bf16-rounded block statistics, the same CSR on both sides.  bf16 tolerances."""
import numpy as np
import pytest
import torch

import oracle
import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu


def gpu_remainder(w, q, k, v, rp, ci, order=0, N=None, scores=None):
    N = w.N if N is None else N
    o = torch.full(v.shape, 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((q.shape[0], q.shape[1], N), 7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = B.make_problem(q, k, v, o, N, w.block)
    ws = torch.full((B.attn_remainder_workspace_bytes(p, order),), 0xFF, dtype=torch.uint8, device="cuda")
    B.block_sparse_attn_remainder_fwd(p, q, k, v, rp, ci, o, lse, status, order, ws, scores)
    torch.cuda.synchronize()
    return o, lse, int(status.item())


def check_vs_oracle(w, qb, kb, vb, rp, ci, o, lse, rows, order=0):
    o_ref, l_ref = oracle.attn_remainder_rows(qb, kb, vb, w.N, w.block, w.scale, rp.cpu().numpy(), ci.cpu().numpy(),
                                              rows, order=order, stats="bf16")
    max_abs, rel, lse_err = U.attn_errors(o, lse, o_ref, l_ref, rows, w.N, w.block, o.shape[1])
    assert max_abs <= U.BF16_MAX_ABS and rel <= U.BF16_REL_L2 and lse_err <= 2e-3, (max_abs, rel, lse_err)
    return max_abs, rel, lse_err


CASES = {
    "medium_h2": shrink(WORKLOADS["medium"], H=2),                                   # Nb = 64: one pooled tile
    "ragged_tail": shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, k=5),         # N = 1860: last block of 68 keys
    "two_pooled_tiles": shrink(WORKLOADS["large"], H=2, T=14, k=20),                 # Nb = 171 > 128
    "mass_ragged_rows": shrink(WORKLOADS["large_ragged"], H=2, T=8),
    "window": shrink(WORKLOADS["xl"], B=2, H=2, T=5),
    "single_block": shrink(WORKLOADS["medium"], H=1, T=1, Hg=8, Wg=16, k=1),         # nothing dropped
    "b64": shrink(WORKLOADS["medium"], H=2, T=2, block=64, k=8),
    "b64_ragged_tail": shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, block=64, k=7),   # 30 blocks, 4-key tail
    "b64_odd_nb": shrink(WORKLOADS["medium"], H=2, T=1, Hg=30, Wg=30, block=64, k=4),        # 15 blocks
    "b64_three_pooled_tiles": shrink(WORKLOADS["large_b64"], H=1, T=11, k=30),               # Nb = 269
}


@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("name", list(CASES))
def test_remainder_matches_oracle(name, order):
    w = CASES[name]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, scores = U.gpu_select(w, qd, kd, want_scores=order == 1)
    o, lse, st = gpu_remainder(w, qd, kd, vd, rp, ci, order, scores=scores)
    assert st == 0
    rows = list(range(w.R)) if w.R <= 160 else U.sample_rows_per_head(w.B * w.H, w.Nb, 6, seed=1)
    r = check_vs_oracle(w, qb, kb, vb, rp, ci, o, lse, rows, order)
    print(f"{name} order {order}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e} lse {r[2]:.2e}")
    if w.n_alloc > w.N:
        assert (o[:, :, w.N:] == 7.0).all()


@pytest.mark.parametrize("name", ["two_pooled_tiles", "ragged_tail", "mass_ragged_rows"])
def test_both_ways_of_masking_the_kept_blocks_agree(name):
    """128-token blocks, at most 1024 key blocks: the K producer leaves the kept blocks of a row as a bit mask in shared
    memory; beyond that the softmax warps look them up in the CSR.  The second form is forced here (debug bit 7) on
    cases the first one serves: same bytes, and the oracle check of the forced form."""
    w = CASES[name]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, scores = U.gpu_select(w, qd, kd, want_scores=True)
    for order in (0, 1):
        o_mask, lse_mask, st = gpu_remainder(w, qd, kd, vd, rp, ci, order, scores=scores)
        assert st == 0
        B.debug_set_mode(128)
        try:
            o_csr, lse_csr, st = gpu_remainder(w, qd, kd, vd, rp, ci, order, scores=scores)
        finally:
            B.debug_set_mode(0)
        assert st == 0
        assert torch.equal(o_mask.view(torch.int16), o_csr.view(torch.int16)) and torch.equal(lse_mask, lse_csr)
        rows = list(range(w.R)) if w.R <= 160 else U.sample_rows_per_head(w.B * w.H, w.Nb, 4, seed=2)
        check_vs_oracle(w, qb, kb, vb, rp, ci, o_csr, lse_csr, rows, order)


@pytest.mark.parametrize("name", ["medium_h2", "b64_odd_nb", "two_pooled_tiles"])
def test_first_order_term_where_it_matters(name):
    """V correlated with K inside every block (v += 4 k), so that C_J = sum (k - kbar) v^T is large and the
    first-order term moves the output by more than twice the tolerance: a missing term, a wrong sign, a transposed C_J or A_I, a wrong
    weight or reference would all fail here (on the plain workloads the term is smaller than the bf16 noise)."""
    from paper_2606_23743_b200.workloads import bf16_bits
    w = CASES[name]
    (q, k, v), (qb, kb, _) = U.host_inputs(w)
    v = (v.float() + 4.0 * k.float()).to(torch.bfloat16)
    vb = bf16_bits(v)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, scores = U.gpu_select(w, qd, kd, want_scores=True)
    o1, lse1, st = gpu_remainder(w, qd, kd, vd, rp, ci, 1, scores=scores)
    assert st == 0
    rows = list(range(w.R)) if w.R <= 160 else U.sample_rows_per_head(w.B * w.H, w.Nb, 6, seed=1)
    rpn, cin = rp.cpu().numpy(), ci.cpu().numpy()
    ref0, _ = oracle.attn_remainder_rows(qb, kb, vb, w.N, w.block, w.scale, rpn, cin, rows, order=0, stats="bf16")
    ref1, l1 = oracle.attn_remainder_rows(qb, kb, vb, w.N, w.block, w.scale, rpn, cin, rows, order=1, stats="bf16")
    ok = ~np.isnan(ref1)
    moved = np.linalg.norm((ref1 - ref0)[ok]) / np.linalg.norm(ref1[ok])
    assert moved > 2 * U.BF16_REL_L2, moved                  # the term is worth more than two tolerances here (a flipped sign: four)
    o0, _, _ = gpu_remainder(w, qd, kd, vd, rp, ci, 0)
    d_gpu = U.attn_errors(o1, None, ref0, l1, rows, w.N, w.block, o1.shape[1])[1]        # rel-L2 of GPU order 1 to oracle order 0
    assert d_gpu > 1.5 * U.BF16_REL_L2, d_gpu                # ... and the GPU's order 1 is not order 0
    max_abs, rel, lse_err = U.attn_errors(o1, lse1, ref1, l1, rows, w.N, w.block, o1.shape[1])
    print(f"{name}: first-order term moves the output by rel-L2 {moved:.3f}; GPU vs oracle rel_l2 {rel:.2e} max_abs {max_abs:.2e}")
    assert rel <= U.BF16_REL_L2 and lse_err <= 2e-3
    assert max_abs <= max(U.BF16_MAX_ABS, 2.0 ** -7 * float(np.nanmax(np.abs(ref1))))     # (outputs of magnitude > 2.5: one bf16 unit)


def test_rows_that_drop_nothing_equal_the_exact_call_and_empty_rows_are_all_remainder():
    w = shrink(WORKLOADS["medium"], H=2, T=2, k=3)           # Nb = 16
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, _ = U.gpu_select(w, qd, kd)
    rp_h, ci_h = rp.cpu(), ci.cpu()
    kept = [ci_h[rp_h[r]:rp_h[r + 1]].tolist() for r in range(w.R)]
    kept[2] = list(range(w.Nb))                              # keeps everything: no remainder
    kept[5] = []                                             # keeps nothing: the remainder is the whole answer
    kept[w.R - 1] = list(range(w.Nb))
    rp2 = torch.zeros(w.R + 1, dtype=torch.int32); rp2[1:] = torch.cumsum(torch.tensor([len(x) for x in kept]), 0)
    ci2 = torch.tensor([j for x in kept for j in x], dtype=torch.int32)
    o, lse, st = gpu_remainder(w, qd, kd, vd, rp2.cuda(), ci2.cuda())
    assert st == 0
    check_vs_oracle(w, qb, kb, vb, rp2, ci2, o, lse, list(range(w.R)))
    o_e, lse_e, _ = U.gpu_attn(w, qd, kd, vd, rp2.cuda(), ci2.cuda())
    for r in (2, w.R - 1):
        bh, I = divmod(r, w.Nb)
        sl = (bh // w.H, bh % w.H, slice(I * w.block, min((I + 1) * w.block, w.N)))
        assert torch.equal(o[sl], o_e[sl]) and torch.equal(lse[sl], lse_e[sl])


@pytest.mark.parametrize("block", [128, 64])
def test_bad_csr_entries_are_reported_not_trapped(block):
    """An out-of-range col_idx entry and a corrupt row_ptr pair under the remainder (both orders): flagged in
    device_status, nothing faults, rows that the damage does not touch still match the oracle."""
    w = shrink(WORKLOADS["medium"], H=2, T=2, k=3, block=block)
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, scores = U.gpu_select(w, qd, kd, want_scores=True)
    rp_h = rp.cpu()
    ci_bad = ci.clone(); ci_bad[int(rp_h[5])] = 9999
    rp_bad = rp_h.clone(); rp_bad[9] = int(rp_h[8]) - 3                      # not monotone
    for order in (0, 1):
        for rpx, cix, touched in ((rp, ci_bad, {4, 5}), (rp_bad.cuda(), ci, {8, 9})):
            o, lse, st = gpu_remainder(w, qd, kd, vd, rpx, cix, order, scores=scores)
            assert st & B.SVA_DEV_BAD_INDEX and not (st & B.SVA_DEV_TIMEOUT)
            rows = [r for r in range(w.R) if r not in touched and (r ^ 1) not in touched][:10]
            check_vs_oracle(w, qb, kb, vb, rp, ci, o, lse, rows, order)


def test_unsupported_forms_are_refused_on_the_host():
    w = shrink(WORKLOADS["tiny"], H=2)                        # d = 64
    (q, k, v), _ = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, _ = U.gpu_select(w, qd, kd)
    p = B.make_problem(qd, kd, vd, torch.empty_like(vd), w.N, w.block)
    assert B.attn_remainder_workspace_bytes(p) == 0
    with pytest.raises(B.SvaError) as e:
        B.block_sparse_attn_remainder_fwd(p, qd, kd, vd, rp, ci, torch.empty_like(vd), None, None, 0,
                                          torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 2
    w2 = shrink(WORKLOADS["medium"], H=1, T=2)
    (q, k, v), _ = U.host_inputs(w2)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    rp, ci, _ = U.gpu_select(w2, qd, kd)
    p2 = B.make_problem(qd, kd, vd, torch.empty_like(vd), w2.N, w2.block)
    ws = torch.empty(B.attn_remainder_workspace_bytes(p2), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SvaError) as e:                      # first-order term without the score matrix
        B.block_sparse_attn_remainder_fwd(p2, qd, kd, vd, rp, ci, torch.empty_like(vd), None, None, 1, ws)
    assert e.value.status == 1
    with pytest.raises(B.SvaError) as e:                      # the exact call's workspace is too small
        B.block_sparse_attn_remainder_fwd(p2, qd, kd, vd, rp, ci, torch.empty_like(vd), None, None, 0,
                                          ws[: B.attn_one_call_workspace_bytes(p2)])
    assert e.value.status == 3
    with pytest.raises(B.SvaError) as e:                      # order 1 needs more than order 0's workspace
        sc = torch.zeros(w2.B, w2.H, w2.Nb, w2.Nb, dtype=torch.float32, device="cuda")
        B.block_sparse_attn_remainder_fwd(p2, qd, kd, vd, rp, ci, torch.empty_like(vd), None, None, 1, ws, sc)
    assert e.value.status == 3


@pytest.mark.parametrize("seed", [3, 4])
def test_random_configurations_of_the_remainder(seed):
    """Seeded random small shapes (both block sizes, top-k and mass rule, one to nine kept blocks), orders 0 and 1,
    against the oracle.  Order 0 stays inside the convex hull of V and meets the workloads' bounds (2e-2, or one
    bf16 unit of the largest output where a peaked row returns a single V row of magnitude ~4.5).  The first-order
    term is not bounded: where a query block drops almost everything its corrected output leaves the hull (|o| up to
    ~90 for |v| <= 5) as a difference of large terms, each of whose bf16 factors (C_J, weights, A_I, P') rounds once
    -- there the bound is 2 % of the largest output and rel-L2 1e-2 (seen: up to 1.3 % and 8.2e-3); what is checked is
    that the device gives what the formula gives."""
    rng = np.random.default_rng(seed)
    for case in range(24):
        block = int(rng.choice([64, 128]))
        Hh, Bb = int(rng.integers(1, 3)), int(rng.integers(1, 3))
        Hg, Wg, T = int(rng.integers(2, 20)), int(rng.integers(8, 48)), int(rng.integers(1, 8))
        w = shrink(WORKLOADS["medium"], B=Bb, H=Hh, T=T, Hg=Hg, Wg=Wg, block=block, d=128, mode=int(rng.integers(0, 2)),
                   k=int(rng.integers(1, 10)), tau=float(rng.choice([0.5, 0.9, 0.99])), win_t=-1, win_s=-1,
                   sigma_f=float(rng.choice([0.3, 0.65, 1.0])), qk_mult=float(rng.choice([1.0, 1.5])))
        what = f"seed {seed} case {case}: {w}"
        (q, k, v), (qb, kb, vb) = U.host_inputs(w, seed=2000 * seed + case)
        qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
        rp, ci, scores = U.gpu_select(w, qd, kd, want_scores=True)
        rows = list(range(w.R)) if w.R <= 32 else sorted(set(rng.choice(w.R, 32, replace=False).tolist()) | {0, w.R - 1})
        for order in (0, 1):
            o, lse, st = gpu_remainder(w, qd, kd, vd, rp, ci, order, scores=scores)
            assert st == 0, what
            o_ref, l_ref = oracle.attn_remainder_rows(qb, kb, vb, w.N, w.block, w.scale, rp.cpu().numpy(),
                                                      ci.cpu().numpy(), rows, order=order, stats="bf16")
            max_abs, rel, lse_err = U.attn_errors(o, lse, o_ref, l_ref, rows, w.N, w.block, o.shape[1])
            mag = float(np.nanmax(np.abs(o_ref)))
            unit = 2.0 ** (np.floor(np.log2(max(mag, 1e-30))) - 7)                     # one bf16 unit at the largest output
            abs_tol = max(U.BF16_MAX_ABS, unit if order == 0 else 0.02 * mag)
            rel_tol = U.BF16_REL_L2 if order == 0 else 1e-2
            assert max_abs <= abs_tol and rel <= rel_tol and lse_err <= 2e-3, (what, order, max_abs, rel, lse_err, mag)
            if order == 0:
                vmax = float(np.abs(oracle.bf16_to_f64(vb)).max())
                assert mag <= 1.01 * vmax, (what, mag, vmax)                             # inside the hull of V
