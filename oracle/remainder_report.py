"""How far piecewise attention is from DENSE attention with and without the approximate remainder, from the
oracle alone (fp64, sampled query blocks of full-size workloads):  python -m oracle.remainder_report [workload ...]

Prints, per workload, the relative L2 distance to dense attention of (a) exact attention over the kept blocks
only, (b) plus the order-0 remainder, (c) plus the first-order term (collapsed weight), and the share of the
softmax mass the kept blocks hold.  Calls nothing outside oracle/ and the seeded input recipes."""
import sys

import numpy as np

import oracle
from paper_2606_23743_b200.workloads import WORKLOADS, bf16_bits, make_qkv, shrink


def report(name: str, heads: int = 2, rows_per_head: int = 4):
    w = shrink(WORKLOADS[name], B=1, H=heads)
    q, k, v = make_qkv(w)
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    sel, _ = oracle.select_from_qk(qb, kb, w.N, w.block, w.scale, w.mode, w.k, w.tau, w.win_t, w.win_s,
                                   w.blocks_per_frame if w.win_t >= 0 else 0)
    rng = np.random.default_rng(0)
    rows = sorted({h * w.Nb + int(I) for h in range(heads) for I in [0, w.Nb - 1, *rng.integers(0, w.Nb, rows_per_head - 2)]})
    o_d, lse_d = oracle.dense_attn_rows(qb, kb, vb, w.N, w.block, w.scale, rows=rows)
    o_e, lse_e = oracle.attn_rows(qb, kb, vb, w.N, w.block, w.scale, sel.row_ptr, sel.col_idx, rows=rows)
    ok = ~np.isnan(o_d)
    den = np.linalg.norm(o_d[ok])
    out = {"kept blocks only": np.linalg.norm((o_e - o_d)[ok]) / den}
    for order in (0, 1):
        o_r, _ = oracle.attn_remainder_rows(qb, kb, vb, w.N, w.block, w.scale, sel.row_ptr, sel.col_idx, rows, order=order)
        out[f"+ remainder, order {order}"] = np.linalg.norm((o_r - o_d)[ok]) / den
    okl = ~np.isnan(lse_d)
    mass = float(np.exp(lse_e[okl] - lse_d[okl]).mean())
    print(f"{name}: {len(rows)} query blocks of {heads} heads, kept blocks hold {mass:.3f} of the softmax mass on average")
    for key, val in out.items():
        print(f"    {key:26s} rel-L2 to dense attention {val:.4f}")
    return out


if __name__ == "__main__":
    for n in (sys.argv[1:] or ["large", "large_b64"]):
        report(n)
