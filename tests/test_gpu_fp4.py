"""The block-scaled 4-bit path through the C ABI: the quantiser's bytes against the oracle's, bit for bit."""
import numpy as np
import pytest
import torch

import _util as U
from oracle import nvfp4
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

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
        qb = U.bf16_bits(q) if hasattr(U, "bf16_bits") else qb
    from paper_2606_23743_b200.workloads import bf16_bits
    qb = bf16_bits(q)
    q4, k4, qsf, ksf, qg, kg = gpu_quantize4(w, U.dev(q), U.dev(k))
    for bits, g4, gsf, gg in ((qb, q4, qsf, qg), (kb, k4, ksf, kg)):
        codes, sfs, g = nvfp4.quantize(bits, w.N)
        np.testing.assert_array_equal(gg.cpu().numpy().reshape(w.B, w.H), g)
        np.testing.assert_array_equal(untile_sf(gsf, w.Nb).reshape(w.B, w.H, w.Nb * 128, 8), sfs)
        np.testing.assert_array_equal(g4.cpu().numpy().reshape(w.B, w.H, w.Nb * 128, 64), codes)
