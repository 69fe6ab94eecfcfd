"""The seeded input recipes: shapes, determinism, tail, and the structure they promise."""
import numpy as np
import torch

import oracle
from paper_2606_23743_b200.workloads import WORKLOADS, bf16_bits, make_qkv, shrink


def test_sizes_match_the_config_table():
    w = WORKLOADS
    assert (w["tiny"].N, w["tiny"].Nb, w["tiny"].R) == (1024, 16, 32)
    assert (w["medium"].N, w["medium"].Nb, w["medium"].R) == (8192, 64, 1024)
    assert (w["large"].N, w["large"].Nb, w["large"].n_alloc, w["large"].R) == (32760, 256, 32768, 6144)
    assert (w["xl"].N, w["xl"].Nb, w["xl"].R, w["xl"].blocks_per_frame) == (47616, 372, 23808, 12)
    assert w["large_fp8"].fp8 and w["large_fp8"].N == 32760


def test_deterministic_and_tail_zero():
    w = shrink(WORKLOADS["large"], H=1, T=1)          # N = 1560 = 12*128 + 24
    a = make_qkv(w)
    b = make_qkv(w)
    for x, y in zip(a, b):
        assert x.dtype == torch.bfloat16 and x.shape == (1, 1, w.n_alloc, 128)
        assert torch.equal(x, y)
        assert (x[:, :, w.N:] == 0).all() and (x[:, :, :w.N].float().abs().sum() > 0)
    c = make_qkv(w, seed=1)
    assert not torch.equal(a[0], c[0])


def test_same_frame_blocks_score_higher():
    w = WORKLOADS["tiny"]
    q, k, _ = make_qkv(w)
    sel, s = oracle.select_from_qk(bf16_bits(q), bf16_bits(k), w.N, w.block, w.scale, 0, w.k)
    bpf = w.blocks_per_frame
    assert bpf == 4
    for r in range(w.R):
        I = r % w.Nb
        frame = set(range(I // bpf * bpf, I // bpf * bpf + bpf))
        assert set(sel.kept(r).tolist()) == frame          # top-4 == the query's own frame
    assert sel.score_gap.min() > 0.5
