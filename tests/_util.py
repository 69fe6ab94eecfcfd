"""Shared helpers of the GPU parity tests: run the C ABI through the binding, run the oracle on
the same bits, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import Workload, bf16_bits, make_qkv

BF16_MAX_ABS, BF16_REL_L2, FP8_REL_L2 = 2e-2, 1e-2, 5e-2
NEAR_TIE = 1e-4


def dev(x):
    return x.cuda(non_blocking=False)


def gpu_select(w: Workload, q, k, N=None, want_scores=False, q_scale=None, k_scale=None, fp8=False):
    """Runs sva_block_select; returns (row_ptr, col_idx[:nnz], scores|None) as device tensors."""
    N = w.N if N is None else N
    p = B.make_problem(q, k, None, None, N, w.block, 0.0, fp8)
    s = B.make_select(w.mode, w.k, w.tau, w.win_t, w.win_s, w.blocks_per_frame if w.win_t >= 0 else 0)
    Nb = -(-N // w.block)
    R = q.shape[0] * q.shape[1] * Nb
    ws = torch.full((max(B.select_workspace_bytes(p, s), 256),), 0xFF, dtype=torch.uint8, device="cuda")
    row_ptr = torch.full((R + 1,), -7, dtype=torch.int32, device="cuda")
    col_idx = torch.full((max(B.select_max_nnz(p, s), 1),), -7, dtype=torch.int32, device="cuda")
    scores = torch.empty(q.shape[0], q.shape[1], Nb, Nb, dtype=torch.float32, device="cuda") if want_scores else None
    B.block_select(p, s, q, k, row_ptr, col_idx, ws, q_scale, k_scale, scores)
    torch.cuda.synchronize()
    nnz = int(row_ptr[-1].item())
    return row_ptr, col_idx[:nnz], scores


def oracle_select(w: Workload, qb, kb, N=None):
    N = w.N if N is None else N
    return oracle.select_from_qk(qb, kb, N, w.block, w.scale, w.mode, w.k, w.tau, w.win_t, w.win_s,
                                 w.blocks_per_frame if w.win_t >= 0 else 0)


def compare_selection(sel: "oracle.Selection", row_ptr, col_idx):
    """Bit-exact comparison of kept sets; rows that differ must be near-ties of the oracle.
    Returns (n_rows_differing, n_near_tie_rows)."""
    rp = row_ptr.cpu().numpy()
    ci = col_idx.cpu().numpy()
    R = sel.counts.size
    assert rp[0] == 0 and (np.diff(rp) >= 0).all()
    near = (sel.score_gap < NEAR_TIE) | (sel.mass_margin < NEAR_TIE)
    diff_rows = []
    same_counts = np.diff(rp) == sel.counts
    if same_counts.all() and np.array_equal(ci, sel.col_idx):
        return 0, int(near.sum())
    for r in range(R):
        got = ci[rp[r]:rp[r + 1]]
        assert (np.diff(got) > 0).all(), f"row {r} not ascending/unique"
        if not np.array_equal(got, sel.kept(r)):
            diff_rows.append(r)
    bad = [r for r in diff_rows if not near[r]]
    assert not bad, f"{len(bad)} rows differ outside near-ties, first: row {bad[0]} gpu={ci[rp[bad[0]]:rp[bad[0]+1]]} oracle={sel.kept(bad[0])} gap={sel.score_gap[bad[0]]} margin={sel.mass_margin[bad[0]]}"
    return len(diff_rows), int(near.sum())


def gpu_attn(w: Workload, q, k, v, row_ptr, col_idx, N=None, simt=False, dense=False, want_lse=True,
             q_scale=None, k_scale=None, fp8=False):
    N = w.N if N is None else N
    o = torch.full(v.shape, 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((q.shape[0], q.shape[1], N), 7.0, dtype=torch.float32, device="cuda") if want_lse else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = B.make_problem(q, k, v, o, N, w.block, 0.0, fp8)
    # (0xff bytes are NaNs as bf16: whatever the kernels do not write themselves shows up in the output)
    ws = torch.full((max(B.attn_one_call_workspace_bytes(p), 256),), 0xFF, dtype=torch.uint8, device="cuda")
    if dense and not simt:
        B.dense_attn_fwd(p, q, k, v, o, lse, status, q_scale, k_scale, workspace=ws)
    else:
        B.block_sparse_attn_fwd(p, q, k, v, None if dense else row_ptr, None if dense else col_idx, o, lse,
                                status, q_scale, k_scale, simt=simt, workspace=ws)
    torch.cuda.synchronize()
    return o, lse, int(status.item())


def sample_rows(R: int, Nb: int, n: int, seed: int = 0):
    """Always the first row, the last (ragged) block of some head, plus random rows."""
    rng = np.random.default_rng(seed)
    rows = {0, Nb - 1, R - 1}
    while len(rows) < min(n, R):
        rows.add(int(rng.integers(0, R)))
    return sorted(rows)


def sample_rows_per_head(BH: int, Nb: int, n_random: int = 8, seed: int = 0):
    """The full-size sample: for EVERY (b, h) query block 0, the last (ragged) query block and
    `n_random` seeded random ones, as row indices r = bh * Nb + I."""
    rng = np.random.default_rng(seed)
    rows = []
    for bh in range(BH):
        mine = {0, Nb - 1}
        while len(mine) < min(n_random + 2, Nb):
            mine.add(int(rng.integers(0, Nb)))
        rows += [bh * Nb + I for I in sorted(mine)]
    return rows


def attn_errors(o_gpu, lse_gpu, o_ref, lse_ref, rows, N, block, H):
    """o_gpu [B,H,n_alloc,d] bf16 device; o_ref [n_rows, block, d] f64 with NaN for absent queries."""
    Bq, Hq, n_alloc, d = o_gpu.shape
    Nb = -(-N // block)
    # only the sampled query blocks leave the device (a full-size tensor in fp64 would be gigabytes)
    rt = torch.as_tensor(rows, device=o_gpu.device, dtype=torch.int64)
    tok = ((rt % Nb) * block)[:, None] + torch.arange(block, device=o_gpu.device)[None, :]
    flat = o_gpu.reshape(Bq * Hq, n_alloc, d)
    og_rows = flat[(rt // Nb)[:, None], tok.clamp_(max=n_alloc - 1)].float().cpu().numpy().astype(np.float64)
    num = den = 0.0
    max_abs = 0.0
    lse_err = 0.0
    for t, r in enumerate(rows):
        bh, I = divmod(r, Nb)
        lo, hi = I * block, min((I + 1) * block, N)
        ref = o_ref[t, : hi - lo]
        got = og_rows[t, : hi - lo]
        assert not np.isnan(ref).any()
        diff = got - ref
        num += (diff ** 2).sum(); den += (ref ** 2).sum()
        max_abs = max(max_abs, float(np.abs(diff).max()))
        if lse_gpu is not None:
            lg = lse_gpu[bh // Hq, bh % Hq, lo:hi].cpu().numpy().astype(np.float64)
            lse_err = max(lse_err, float(np.abs(lg - lse_ref[t, : hi - lo]).max()))
    return max_abs, float(np.sqrt(num / max(den, 1e-300))), lse_err


def check_attn_vs_oracle(w, qb, kb, vb, row_ptr, col_idx, o_gpu, lse_gpu, rows, N=None, dense=False,
                         rel_tol=BF16_REL_L2, abs_tol=BF16_MAX_ABS):
    N = w.N if N is None else N
    if dense:
        o_ref, l_ref = oracle.dense_attn_rows(qb, kb, vb, N, w.block, w.scale, rows=rows)
    else:
        o_ref, l_ref = oracle.attn_rows(qb, kb, vb, N, w.block, w.scale, row_ptr.cpu().numpy(),
                                        col_idx.cpu().numpy(), rows=rows)
    max_abs, rel, lse_err = attn_errors(o_gpu, lse_gpu, o_ref, l_ref, rows, N, w.block, o_gpu.shape[1])
    assert max_abs <= abs_tol, f"max-abs {max_abs} > {abs_tol}"
    assert rel <= rel_tol, f"rel-L2 {rel} > {rel_tol}"
    if lse_gpu is not None:
        assert lse_err <= 2e-3, f"lse err {lse_err}"
    return max_abs, rel, lse_err


def host_inputs(w: Workload, seed=None):
    q, k, v = make_qkv(w, seed)
    return (q, k, v), (bf16_bits(q), bf16_bits(k), bf16_bits(v))


def oracle_fp8_inputs(w: Workload, qb, kb, q8, k8, qs, ks):
    """What the oracle is run on in the FP8 tests: its own codes and scales, made from the bf16 inputs and
    dequantised in fp64.  The GPU quantiser's bytes must equal them, so the two sides see the same Q, K and
    nothing the oracle consumes comes from the CUDA path."""
    out = []
    for bits, g8, gs in ((qb, q8, qs), (kb, k8, ks)):
        codes, scales = oracle.quantize_e4m3(bits, w.N, w.block)
        np.testing.assert_array_equal(gs.cpu().numpy(), scales)
        assert np.array_equal(g8.cpu().numpy()[:, :, :w.N], codes[:, :, :w.N])
        out.append(oracle.dequantize_e4m3(codes, scales, w.N, w.block))
    return out
