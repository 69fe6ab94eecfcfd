"""The block-scaled 4-bit path through the C ABI: the quantiser's bytes against the oracle's, bit for bit."""
import numpy as np
import pytest
import torch

import _util as U
from oracle import nvfp4
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, bf16_bits, shrink

pytestmark = pytest.mark.gpu


def gpu_quantize4(w, qd, kd):
    BH = w.B * w.H
    q4 = torch.full((BH, w.Nb * 128, 64), 0xAB, dtype=torch.uint8, device="cuda"); k4 = q4.clone()
    qsf = torch.full((BH, w.Nb, 1024), 0xAB, dtype=torch.uint8, device="cuda"); ksf = qsf.clone()
    qg = torch.zeros(BH, dtype=torch.float32, device="cuda"); kg = torch.zeros_like(qg)
    ws = torch.full((max(8 * BH, 256),), 0xFF, dtype=torch.uint8, device="cuda")
    p = B.make_problem(qd, kd, None, None, w.N, w.block)
    B.quantize_qk_fp4(p, qd, kd, q4, k4, qsf, ksf, qg, kg, ws)
    torch.cuda.synchronize()
    return q4, k4, qsf, ksf, qg, kg


def untile_sf(sf_tiled, Nb):
    """[BH][Nb][2][32][4][4] bytes -> [BH][Nb*128 tokens][8 scale blocks]."""
    x = sf_tiled.cpu().numpy().reshape(-1, Nb, 2, 32, 4, 4)        # [bh, I, half, t%32, t/32, kb]
    x = x.transpose(0, 1, 4, 3, 2, 5)                               # [bh, I, t/32, t%32, half, kb]
    return x.reshape(x.shape[0], Nb * 128, 8)


@pytest.mark.parametrize("name", ["medium_h3", "ragged"])
def test_quantiser_bytes_equal_the_oracle(name):
    w = {"medium_h3": shrink(WORKLOADS["medium"], H=3, T=2),
         "ragged": shrink(WORKLOADS["large"], H=2, T=1)}[name]                       # N = 1560: a 24-token last block
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    if name == "ragged":
        q[0, 1, 5] = 0                                                               # an all-zero token: scales 0, codes 0
    qb = bf16_bits(q)
    q4, k4, qsf, ksf, qg, kg = gpu_quantize4(w, U.dev(q), U.dev(k))
    for bits, g4, gsf, gg in ((qb, q4, qsf, qg), (kb, k4, ksf, kg)):
        codes, sfs, g = nvfp4.quantize(bits, w.N)
        np.testing.assert_array_equal(gg.cpu().numpy().reshape(w.B, w.H), g)
        np.testing.assert_array_equal(untile_sf(gsf, w.Nb).reshape(w.B, w.H, w.Nb * 128, 8), sfs)
        np.testing.assert_array_equal(g4.cpu().numpy().reshape(w.B, w.H, w.Nb * 128, 64), codes)


# Against the oracle run on the DEQUANTISED Q, K the 4-bit path is as exact as the bf16 one (products of e2m1 codes
# and e4m3 scales are exact in the MMA's fp32 accumulation): the bf16 bar applies.
FP4_REL_L2, FP4_MAX_ABS = U.BF16_REL_L2, U.BF16_MAX_ABS


def gpu_attn_fp4(w, quant, vd, rp, ci):
    q4, k4, qsf, ksf, qg, kg = quant
    o = torch.full(vd.shape, 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.B, w.H, w.N), 7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = B.make_problem(vd, vd, vd, o, w.N, w.block)
    ws = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")          # the row counters: V is read where it lies
    B.block_sparse_attn_fwd_fp4(p, q4, k4, qsf, ksf, qg, kg, vd, rp, ci, o, lse, status, ws)
    torch.cuda.synchronize()
    return o, lse, int(status.item())


def oracle_dequantised(w, qb, kb):
    return tuple(nvfp4.dequantize(*nvfp4.quantize(bits, w.N)) for bits in (qb, kb))


@pytest.mark.parametrize("name", ["two_blocks_dense", "medium_h2", "ragged_tail", "mass_rows"])
def test_fp4_attention_matches_oracle_on_dequantised_inputs(name):
    w = {"two_blocks_dense": shrink(WORKLOADS["medium"], H=1, T=1, Hg=16, Wg=16, k=2),       # N = 256, keep-all
         "medium_h2": shrink(WORKLOADS["medium"], H=2),
         "ragged_tail": shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, k=5),
         "mass_rows": shrink(WORKLOADS["large_ragged"], H=2, T=8)}[name]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    quant = gpu_quantize4(w, qd, kd)
    qh, kh = oracle_dequantised(w, qb, kb)                       # (the GPU quantiser's bytes equal the oracle's: tested above)
    sel, _ = U.oracle_select(w, qh, kh)
    rp = torch.from_numpy(sel.row_ptr).cuda(); ci = torch.from_numpy(sel.col_idx).cuda()
    o, lse, st = gpu_attn_fp4(w, quant, vd, rp, ci)
    assert st == 0
    rows = list(range(w.R)) if w.R <= 128 else U.sample_rows_per_head(w.B * w.H, w.Nb, 6, seed=2)
    r = U.check_attn_vs_oracle(w, qh, kh, vb, rp, ci, o, lse, rows, rel_tol=FP4_REL_L2, abs_tol=FP4_MAX_ABS)
    print(f"{name}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e} lse {r[2]:.2e}")
    if name == "two_blocks_dense":
        od, lsed, st = gpu_attn_fp4(w, quant, vd, None, None)
        assert st == 0
        U.check_attn_vs_oracle(w, qh, kh, vb, None, None, od, lsed, rows, dense=True, rel_tol=FP4_REL_L2, abs_tol=FP4_MAX_ABS)


def test_fp4_full_size_and_distance_to_bf16_attention():
    """cfg-3 tokens, 4-bit Q/K, in the launch configuration `bench.py --fp4` times: per-head sample against the
    oracle on the dequantised inputs; and, reported, how far 4-bit attention is from bf16 attention on the same CSR."""
    w = WORKLOADS["large"]
    (q, k, v), (qb, kb, vb) = U.host_inputs(w)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    quant = gpu_quantize4(w, qd, kd)
    rp, ci, _ = U.gpu_select(w, qd, kd)                     # routing on the bf16 Q, K
    o, lse, st = gpu_attn_fp4(w, quant, vd, rp, ci)
    assert st == 0
    heads = [0, 7, 23]                                      # the oracle quantiser is numpy: three heads' worth of it
    qh, kh = (nvfp4.dequantize(*nvfp4.quantize(bits[:, heads], w.N)) for bits in (qb, kb))
    for t, h in enumerate(heads):
        sl = slice(h * w.Nb, (h + 1) * w.Nb)
        rp_h = (rp[h * w.Nb:(h + 1) * w.Nb + 1] - rp[h * w.Nb]).cpu()
        ci_h = ci[int(rp[h * w.Nb]):int(rp[(h + 1) * w.Nb])].cpu()
        rows = U.sample_rows_per_head(1, w.Nb, 8, seed=h)
        w1 = shrink(w, H=1)
        r = U.check_attn_vs_oracle(w1, qh[:, t:t + 1], kh[:, t:t + 1], vb[:, h:h + 1], rp_h, ci_h, o[:, h:h + 1], lse[:, h:h + 1],
                                   rows, rel_tol=FP4_REL_L2, abs_tol=FP4_MAX_ABS)
        print(f"large fp4 head {h}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e} lse {r[2]:.2e}")
    o16, _, _ = U.gpu_attn(w, qd, kd, vd, rp, ci)
    a, b = o[:, :, :w.N].float(), o16[:, :, :w.N].float()
    print(f"4-bit vs bf16 attention on the same CSR: rel_l2 {float(torch.linalg.vector_norm(a - b) / torch.linalg.vector_norm(b)):.3f}")
    assert torch.isfinite(a).all()
