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


def test_tile_list_start_formula_leaves_room_for_every_earlier_row():
    """64-token blocks: tile row t's descriptors start at ceil((CSR entries before it + t) / 2) -- no scan.
    Every earlier tile row s needs ceil(|A_s u B_s| / 2) <= ceil((|A_s| + |B_s|) / 2) tiles; the starts must
    leave at least that much room, for any row lengths, and stay below the capacity the workspace reserves."""
    import numpy as np
    rng = np.random.default_rng(7)
    for Nb in (1, 2, 7, 16, 33):
        for _ in range(50):
            H = int(rng.integers(1, 4))
            R = H * Nb
            counts = rng.integers(0, Nb + 1, size=R)
            row_ptr = np.concatenate([[0], np.cumsum(counts)])
            Nt = (Nb + 1) // 2
            starts, need = [], []
            for t in range(H * Nt):
                bh, I2 = divmod(t, Nt)
                rA = bh * Nb + 2 * I2
                a = counts[rA]
                b = counts[rA + 1] if 2 * I2 + 1 < Nb else 0
                starts.append((row_ptr[rA] + t + 1) // 2)
                need.append((a + b + 1) // 2)          # worst case: disjoint lists
            for t in range(len(starts) - 1):
                assert starts[t] + need[t] <= starts[t + 1]
            cap = (R * Nb + H * Nt) // 2 + 2
            assert starts[-1] + need[-1] <= cap
