"""Selection parity through the C ABI: kept sets bit-exact against the fp64 oracle (rows that
differ must be oracle near-ties, which are counted), CSR well-formed, scores within fp32 error."""
import numpy as np
import pytest
import torch

import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu

CASES = {
    "tiny": WORKLOADS["tiny"],
    "medium": WORKLOADS["medium"],
    "ragged_tail": shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, k=5),        # N = 1860
    "mass": shrink(WORKLOADS["large"], H=4, T=8),                                    # cap binds
    "mass_ragged_rows": shrink(WORKLOADS["large_ragged"], H=4, T=8),                 # variable counts
    "window": shrink(WORKLOADS["xl"], B=2, H=2, T=6),                                # 3x3 forced, k=37
    "window_gt_k": shrink(WORKLOADS["xl"], B=1, H=2, T=4, k=5),                      # |F| up to 9 > k
    "window_mass": shrink(WORKLOADS["xl"], B=1, H=2, T=4, mode=1, k=20, tau=0.5),
    "block64_d128": shrink(WORKLOADS["medium"], H=2, T=2, block=64, k=8),
    "k_ge_nb": shrink(WORKLOADS["tiny"], k=99),
    "k1": shrink(WORKLOADS["medium"], H=2, T=2, k=1),
}


@pytest.mark.parametrize("name", list(CASES))
def test_selection_matches_oracle(name):
    w = CASES[name]
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    rp, ci, sc = U.gpu_select(w, U.dev(q), U.dev(k), want_scores=True)
    sel, s_ref = U.oracle_select(w, qb, kb)
    assert np.abs(sc.cpu().numpy() - s_ref).max() < 2e-5
    assert int(rp[-1]) == ci.numel()
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    print(f"{name}: rows {w.R} differing {n_diff} near-tie rows {n_near}")
    assert n_diff <= n_near


def test_exact_ties_resolve_to_lower_index():
    """Blocks with identical tokens give exactly equal scores on the GPU too."""
    w = shrink(WORKLOADS["medium"], H=1, T=2, k=3)        # Nb = 16
    g = torch.Generator().manual_seed(1)
    base = torch.randint(-2, 3, (4, w.d), generator=g).float()
    pat = torch.tensor([0, 1, 2, 3, 0, 1, 2, 3, 3, 2, 1, 0, 0, 0, 1, 1])
    x = base[pat].repeat_interleave(w.block, 0)[None, None].bfloat16().contiguous()
    rp, ci, sc = U.gpu_select(w, U.dev(x), U.dev(x), want_scores=True)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    sel, s_ref = U.oracle_select(w, bits, bits)
    assert (sel.score_gap == 0).any()                     # the case really has boundary ties
    g = sc.cpu().numpy()
    np.testing.assert_allclose(g, s_ref, rtol=1e-6)
    assert g[0, 0, 0, 0] == g[0, 0, 0, 4] == g[0, 0, 0, 11]     # equal blocks score exactly equal
    np.testing.assert_array_equal(ci.cpu().numpy(), sel.col_idx)


def test_strided_views_and_determinism():
    w = shrink(WORKLOADS["medium"], H=2, T=2)
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    qkv = torch.zeros(w.B, w.n_alloc, 2, w.H, w.d, dtype=torch.bfloat16, device="cuda")   # packed [B,N,2,H,d]
    qkv[:, :, 0] = U.dev(q).permute(0, 2, 1, 3)
    qkv[:, :, 1] = U.dev(k).permute(0, 2, 1, 3)
    qv, kv = qkv[:, :, 0].permute(0, 2, 1, 3), qkv[:, :, 1].permute(0, 2, 1, 3)
    assert not qv.is_contiguous()
    rp1, ci1, _ = U.gpu_select(w, qv, kv)
    rp2, ci2, _ = U.gpu_select(w, U.dev(q), U.dev(k))
    assert torch.equal(rp1, rp2) and torch.equal(ci1, ci2)
    rp3, ci3, _ = U.gpu_select(w, qv, kv)
    assert torch.equal(ci1, ci3)


def test_workspace_too_small_is_rejected():
    w = CASES["mass"]
    (q, k, _), _ = U.host_inputs(w)
    qd, kd = U.dev(q), U.dev(k)
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    s = B.make_select(w.mode, w.k, w.tau)
    ws = torch.empty(B.select_workspace_bytes(p, s) - 256, dtype=torch.uint8, device="cuda")
    rp = torch.zeros(w.R + 1, dtype=torch.int32, device="cuda")
    ci = torch.zeros(B.select_max_nnz(p, s), dtype=torch.int32, device="cuda")
    with pytest.raises(B.SvaError) as e:
        B.block_select(p, s, qd, kd, rp, ci, ws)
    assert e.value.status == 3


@pytest.mark.parametrize("name", ["medium", "large_fp8"])
def test_routing_in_two_calls_equals_the_one_call(name):
    """sva_pool_qk + sva_block_select_pooled = sva_block_select (bf16 and e4m3 inputs); the means against
    the oracle's pooling."""
    import oracle
    from paper_2606_23743_b200 import binding as B
    from paper_2606_23743_b200.workloads import shrink
    w = shrink(WORKLOADS[name], H=2, T=3)
    (q, k, _), (qb, kb, _) = U.host_inputs(w)
    qd, kd = U.dev(q), U.dev(k)
    qs = ks = None
    if w.fp8:
        q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda"); k8 = torch.zeros_like(q8)
        qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda"); ks = torch.zeros_like(qs)
        B.quantize_qk_fp8(B.make_problem(qd, kd, None, None, w.N, w.block), qd, kd, q8, k8, qs, ks)
        qd, kd = q8, k8
    rp1, ci1, _ = U.gpu_select(w, qd, kd, q_scale=qs, k_scale=ks, fp8=w.fp8)
    p = B.make_problem(qd, kd, None, None, w.N, w.block, 0.0, w.fp8)
    s = B.make_select(w.mode, w.k, w.tau, w.win_t, w.win_s, w.blocks_per_frame if w.win_t >= 0 else 0)
    qm = torch.full((w.B, w.H, w.Nb, w.d), 7.0, dtype=torch.float32, device="cuda"); km = torch.full_like(qm, 7.0)
    B.pool_qk(p, qd, kd, qm, km, qs, ks)
    rp2 = torch.zeros(w.R + 1, dtype=torch.int32, device="cuda")
    ci2 = torch.zeros(B.select_max_nnz(p, s), dtype=torch.int32, device="cuda")
    ws = torch.empty(B.select_workspace_bytes(p, s), dtype=torch.uint8, device="cuda")
    B.block_select_pooled(p, s, qm, km, rp2, ci2, ws)
    torch.cuda.synchronize()
    assert torch.equal(rp1, rp2) and torch.equal(ci1, ci2[: int(rp2[-1])])
    if w.fp8:
        qb, kb = U.oracle_fp8_inputs(w, qb, kb, qd, kd, qs, ks)
    np.testing.assert_allclose(qm.cpu().numpy(), oracle.pool(qb, w.N, w.block), rtol=2e-6, atol=2e-7)
    np.testing.assert_allclose(km.cpu().numpy(), oracle.pool(kb, w.N, w.block), rtol=2e-6, atol=2e-7)


@pytest.mark.parametrize("T,Hg,Wg,mode,k,tau,d", [(25, 40, 40, 0, 20, 1.0, 128), (16, 64, 64, 1, 30, 0.95, 64)])
def test_many_blocks_per_head(T, Hg, Wg, mode, k, tau, d):
    """625 and 1024 (the maximum) 64-token blocks per head: every lane of the selection warp holds up to 32
    scores of its row; routing against the oracle, attention on sampled rows."""
    w = shrink(WORKLOADS["medium"], B=1, H=1, T=T, Hg=Hg, Wg=Wg, block=64, mode=mode, k=k, tau=tau, d=d, win_t=-1, win_s=-1)
    (q, kk, v), (qb, kb, vb) = U.host_inputs(w, seed=5)
    qd, kd, vd = U.dev(q), U.dev(kk), U.dev(v)
    rp, ci, sc = U.gpu_select(w, qd, kd, want_scores=True)
    sel, s_ref = U.oracle_select(w, qb, kb)
    assert np.abs(sc.cpu().numpy() - s_ref).max() < 2e-5
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    o, lse, st = U.gpu_attn(w, qd, kd, vd, rp, ci)
    assert st == 0
    U.check_attn_vs_oracle(w, qb, kb, vb, rp, ci, o, lse, U.sample_rows(w.R, w.Nb, 6))
