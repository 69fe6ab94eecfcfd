"""Attention parity through the C ABI against the fp64 oracle with an identical CSR on both
sides.  Tolerances are the bf16 bar of the problem statement: max-abs <= 2e-2, rel-L2 <= 1e-2."""
import numpy as np
import pytest
import torch

import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu


def _setup(w):
    (q, k, v), bits = U.host_inputs(w)
    data = (U.dev(q), U.dev(k), U.dev(v))
    rp, ci, _ = U.gpu_select(w, data[0], data[1])
    return data, bits, rp, ci


CASES = {
    "tiny_block64": (WORKLOADS["tiny"], None),                                   # d = 64: computed as d = 128 with a zero upper half
    "medium_h4": (shrink(WORKLOADS["medium"], H=4), 10),
    "ragged_tail": (shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, k=5), None),
    "odd_nb": (shrink(WORKLOADS["medium"], H=2, T=1, Hg=30, Wg=30, k=4), None),  # Nb = 8 -> N=900: Nb=8
    "mass_ragged_rows": (shrink(WORKLOADS["large_ragged"], H=2, T=8), 12),
    "window": (shrink(WORKLOADS["xl"], B=2, H=2, T=5), 12),
    "single_block": (shrink(WORKLOADS["medium"], H=1, T=1, Hg=8, Wg=16, k=1), None),   # N = 128
    "short_tail_only": (shrink(WORKLOADS["medium"], H=2, T=1, Hg=5, Wg=20, k=1), None),  # N = 100 < block
    # 64-token blocks with d = 128 run on the tensor-core kernel too (two query blocks and two key blocks per tile)
    "block64_d128": (shrink(WORKLOADS["medium"], H=2, T=2, block=64, k=8), 10),
    "b64_ragged_tail": (shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, block=64, k=7), None),    # N = 1860: 30 blocks, 4-key tail
    "b64_odd_nb": (shrink(WORKLOADS["medium"], H=2, T=1, Hg=30, Wg=30, block=64, k=4), None),       # N = 900: 15 blocks
    "b64_mass_ragged_rows": (shrink(WORKLOADS["large_ragged"], H=2, T=8, block=64, k=60), 14),
    "b64_k1": (shrink(WORKLOADS["medium"], H=2, T=2, block=64, k=1), 12),
    "b64_single_block": (shrink(WORKLOADS["medium"], H=1, T=1, Hg=5, Wg=8, block=64, k=1), None),   # N = 40 < block
    "block128_d64": (shrink(WORKLOADS["tiny"], H=2, T=4, block=128, k=3), None),
    "d64_ragged_tail": (shrink(WORKLOADS["medium"], H=3, T=2, Hg=30, Wg=31, k=5, d=64), None),       # N = 1860, d = 64
    "d64_mass_ragged_rows": (shrink(WORKLOADS["large_ragged"], H=2, T=8, d=64), 12),
    "d64_b64_odd_nb": (shrink(WORKLOADS["medium"], H=2, T=1, Hg=30, Wg=30, block=64, k=4, d=64), None),
    "many_rows_few_blocks": (shrink(WORKLOADS["medium"], H=6, T=8, k=2), 12),            # R = 384 > 148 CTAs, 2 blocks per row
    "one_block_rows": (shrink(WORKLOADS["medium"], H=3, T=4, k=1), 10),                  # odd row length 1: only one group has work
}


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("impl", ["tensor", "simt"])
def test_sparse_attention_matches_oracle(name, impl):
    w, nrows = CASES[name]
    data, bits, rp, ci = _setup(w)
    o, lse, st = U.gpu_attn(w, *data, rp, ci, simt=(impl == "simt"))
    assert st == 0
    rows = list(range(w.R)) if nrows is None else U.sample_rows(w.R, w.Nb, nrows)
    r = U.check_attn_vs_oracle(w, *bits, rp, ci, o, lse, rows)
    print(f"{name}/{impl}: max_abs {r[0]:.2e} rel_l2 {r[1]:.2e} lse {r[2]:.2e}")
    # absent query rows are never written
    if w.n_alloc > w.N:
        assert (o[:, :, w.N:] == 7.0).all()


@pytest.mark.parametrize("name", ["ragged_tail", "medium_h4", "b64_ragged_tail", "b64_odd_nb", "d64_ragged_tail", "d64_b64_odd_nb"])
def test_dense_equals_keep_all_and_oracle(name):
    w, _ = CASES[name]
    data, bits, _, _ = _setup(w)
    o_d, lse_d, st = U.gpu_attn(w, *data, None, None, dense=True)
    assert st == 0
    rows = U.sample_rows(w.R, w.Nb, 6)
    U.check_attn_vs_oracle(w, *bits, None, None, o_d, lse_d, rows, dense=True)
    # keep-ratio 1.0 through the sparse entry point gives the same bytes as the dense one
    wk = shrink(w, mode=0, k=w.Nb)
    rp, ci, _ = U.gpu_select(wk, data[0], data[1])
    assert ci.numel() == w.R * w.Nb
    o_s, lse_s, _ = U.gpu_attn(w, *data, rp, ci)
    assert torch.equal(o_s, o_d) and torch.equal(lse_s, lse_d)


def test_repeatable_bytes():
    """Launches on the same inputs give identical bytes (no atomics, fixed summation order; this is
    also what a race between the warp roles would break)."""
    w, _ = CASES["mass_ragged_rows"]
    data, bits, rp, ci = _setup(w)
    o1, l1, _ = U.gpu_attn(w, *data, rp, ci)
    for _ in range(3):
        o2, l2, _ = U.gpu_attn(w, *data, rp, ci)
        assert torch.equal(o1, o2) and torch.equal(l1, l2)
    wd = shrink(WORKLOADS["medium"], H=2)                 # long rows: 64 blocks each
    data, bits, _, _ = _setup(wd)
    od, ld, _ = U.gpu_attn(wd, *data, None, None, dense=True)
    for _ in range(3):
        o2, l2, _ = U.gpu_attn(wd, *data, None, None, dense=True)
        assert torch.equal(od, o2) and torch.equal(ld, l2)


@pytest.mark.parametrize("name", ["mass_ragged_rows", "b64_mass_ragged_rows", "d64_mass_ragged_rows"])
def test_two_step_form_matches_the_one_call_form(name):
    """V prepared on a second stream, then the attention kernel alone: same bytes as the one-call entry
    points (sparse and, for 128-token blocks, dense), and the workspace can be prepared again for the next call."""
    w, _ = CASES[name]
    (qd, kd, vd), bits, rp, ci = _setup(w)
    o1, l1, st1 = U.gpu_attn(w, qd, kd, vd, rp, ci)
    od, ld, _ = U.gpu_attn(w, qd, kd, vd, None, None, dense=True)
    o2 = torch.full_like(o1, 3.0); l2 = torch.full_like(l1, 3.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = B.make_problem(qd, kd, vd, o2, w.N, w.block)
    ws = torch.full((B.attn_workspace_bytes(p),), 0xFF, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    for sparse in ((True, False, True) if w.block == 128 else (True, True)):
        ready = torch.cuda.Event()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            B.attn_prepare_v(p, vd, ws)
            ready.record()
        torch.cuda.current_stream().wait_event(ready)
        B.block_sparse_attn_fwd_prepared(p, qd, kd, rp if sparse else None, ci if sparse else None, o2, l2, status,
                                         workspace=ws)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref_o, ref_l = (o1, l1) if sparse else (od, ld)
        assert torch.equal(o2[:, :, :w.N], ref_o[:, :, :w.N]) and torch.equal(l2, ref_l)   # rows >= N are never written
        # the prepared workspace serves a second call on the same V
        o2.fill_(3.0); l2.fill_(3.0)
        B.block_sparse_attn_fwd_prepared(p, qd, kd, rp if sparse else None, ci if sparse else None, o2, l2, status,
                                         workspace=ws)
        torch.cuda.synchronize()
        assert torch.equal(o2[:, :, :w.N], ref_o[:, :, :w.N]) and torch.equal(l2, ref_l)


def test_empty_rows_and_bad_indices_are_reported_not_trapped():
    w = shrink(WORKLOADS["medium"], H=1, T=2, k=2)       # Nb = 16
    data, bits, rp, ci = _setup(w)
    rp_h, ci_h = rp.cpu().clone(), ci.cpu().clone()
    # row 3 empty
    cnt = (rp_h[4] - rp_h[3]).item()
    ci2 = torch.cat([ci_h[: rp_h[3]], ci_h[rp_h[4]:]])
    rp2 = rp_h.clone(); rp2[4:] -= cnt
    for simt in (False, True):
        o, lse, st = U.gpu_attn(w, *data, rp2.cuda(), ci2.cuda(), simt=simt)
        assert st == 0
        assert (o[0, 0, 3 * 128:4 * 128] == 0).all() and torch.isinf(lse[0, 0, 3 * 128:4 * 128]).all()
        rows = [0, 2, 4, 15]
        U.check_attn_vs_oracle(w, *bits, rp2, ci2, o, lse, rows)
    # an out-of-range entry in row 5: flagged, other rows still right
    ci3 = ci_h.clone(); ci3[rp_h[5]] = 999
    for simt in (False, True):
        o, lse, st = U.gpu_attn(w, *data, rp, ci3.cuda(), simt=simt)
        assert st & B.SVA_DEV_BAD_INDEX
        U.check_attn_vs_oracle(w, *bits, rp, ci, o, lse, [0, 4, 6, 15])


@pytest.mark.parametrize("block", [128, 64])
def test_corrupt_row_ptr_is_reported_and_no_entry_outside_the_csr_is_read(block):
    """row_ptr pairs that are not monotone, longer than Nb, or that point far beyond the CSR's row_ptr[R]
    entries: the flag is set, the rows that own a bad pair come out empty (zeros, lse = -inf; with 64-token
    blocks the query block that shares the tile too), no col_idx entry at or beyond row_ptr[R] is read (the
    kernels bound every pair by it), and every other row is still right."""
    w = shrink(WORKLOADS["medium"], H=2, T=2, k=3, block=block)
    data, bits, rp, ci = _setup(w)
    rp_h = rp.cpu().clone()
    nnz, Nb = int(rp_h[-1]), w.Nb
    r0 = 5
    cases = {
        "not monotone": lambda x: x.__setitem__(r0 + 1, int(x[r0]) - 2),
        "longer than Nb": lambda x: x.__setitem__(r0 + 1, int(x[r0]) + Nb + 3),
        "far beyond the CSR": lambda x: (x.__setitem__(r0, 1 << 30), x.__setitem__(r0 + 1, (1 << 30) + 2)),
        "negative": lambda x: x.__setitem__(r0, -4),
    }
    for name, corrupt in cases.items():
        rp2 = rp_h.clone(); corrupt(rp2)
        d = torch.diff(rp2)
        bad = [r for r in range(w.R) if rp2[r] < 0 or d[r] < 0 or d[r] > Nb or rp2[r + 1] > nnz]
        assert bad, name
        touched = set()
        for r in range(w.R):                       # rows whose pair differs from the intact CSR
            if rp2[r] != rp_h[r] or rp2[r + 1] != rp_h[r + 1]:
                touched.add(r)
                if block == 64:
                    touched.add(r ^ 1)             # the other query block of its tile row
        for simt in (False, True):
            o, lse, st = U.gpu_attn(w, *data, rp2.cuda(), ci, simt=simt)
            assert st & B.SVA_DEV_BAD_INDEX, (name, simt)
            assert not (st & B.SVA_DEV_TIMEOUT)
            for r in bad:
                bh, I = divmod(r, Nb)
                sl = (bh // w.H, bh % w.H, slice(I * block, min((I + 1) * block, w.N)))
                assert (o[sl] == 0).all() and torch.isinf(lse[sl]).all(), (name, simt, r)
            rows = [r for r in range(w.R) if r not in touched]
            U.check_attn_vs_oracle(w, *bits, rp_h, ci, o, lse, rows[:6] + rows[-6:])


def test_block64_tile_with_one_empty_query_block():
    """64-token blocks: a tile row whose two query blocks keep different key blocks, down to one of them
    keeping nothing, against the CUDA-core kernel and the oracle."""
    w = shrink(WORKLOADS["medium"], H=2, T=2, block=64, k=6)      # Nb = 32
    data, bits, rp, ci = _setup(w)
    rp_h, ci_h = rp.cpu().clone(), ci.cpu().clone()
    cnt = (rp_h[1:] - rp_h[:-1]).clone()
    keep = torch.ones_like(cnt, dtype=torch.bool)
    keep[1::4] = False            # query block B of every other tile row keeps nothing
    keep[6] = False; keep[7] = False   # a whole tile row without work
    keep[8] = False               # query block A empty, B not
    new_cnt = cnt * keep
    rp2 = torch.zeros_like(rp_h); rp2[1:] = torch.cumsum(new_cnt, 0)
    ci2 = torch.cat([ci_h[rp_h[r]: rp_h[r + 1]] for r in range(w.R) if keep[r]])
    o, lse, st = U.gpu_attn(w, *data, rp2.cuda(), ci2.cuda())
    o_s, lse_s, st_s = U.gpu_attn(w, *data, rp2.cuda(), ci2.cuda(), simt=True)
    assert st == 0 and st_s == 0
    for r in range(w.R):
        bh, I = divmod(r, w.Nb)
        sl = (bh // w.H, bh % w.H, slice(I * w.block, min((I + 1) * w.block, w.N)))
        if not keep[r]:
            assert (o[sl] == 0).all() and torch.isinf(lse[sl]).all() and (lse[sl] < 0).all()
    rows = [r for r in range(w.R) if keep[r]][:24]
    U.check_attn_vs_oracle(w, *bits, rp2, ci2, o, lse, rows)
    assert (o.float() - o_s.float()).abs().max() < 2e-2


def test_runs_of_empty_rows_and_no_rows_at_all():
    """The row scheduler finishes rows with an empty list itself: runs of them (between, before and
    after rows with work) and a CSR without any entry must give zeros / -inf and no hang."""
    w = shrink(WORKLOADS["medium"], H=2, T=2, k=3)       # Nb = 16, R = 32
    data, bits, rp, ci = _setup(w)
    rp_h, ci_h = rp.cpu().clone(), ci.cpu().clone()
    keep = [5, 6, 20]                                    # every other row loses its list
    cnt = rp_h[1:] - rp_h[:-1]
    new_cnt = torch.zeros_like(cnt)
    for r in keep:
        new_cnt[r] = cnt[r]
    rp2 = torch.zeros_like(rp_h); rp2[1:] = torch.cumsum(new_cnt, 0)
    ci2 = torch.cat([ci_h[rp_h[r]: rp_h[r + 1]] for r in keep])
    o_ref, lse_ref, _ = U.gpu_attn(w, *data, rp, ci)
    o, lse, st = U.gpu_attn(w, *data, rp2.cuda(), ci2.cuda())
    assert st == 0
    for r in range(w.R):
        bh, I = divmod(r, w.Nb)
        sl = (bh // w.H, bh % w.H, slice(I * w.block, min((I + 1) * w.block, w.N)))
        if r in keep:
            assert torch.equal(o[sl], o_ref[sl]) and torch.equal(lse[sl], lse_ref[sl])
        else:
            assert (o[sl] == 0).all() and torch.isinf(lse[sl]).all() and (lse[sl] < 0).all()
    # no entry at all
    rp0 = torch.zeros_like(rp)
    o, lse, st = U.gpu_attn(w, *data, rp0, ci)
    assert st == 0 and (o[:, :, :w.N] == 0).all() and torch.isinf(lse).all()


def test_strided_qkv_and_output():
    w = shrink(WORKLOADS["medium"], H=2, T=2)
    (q, k, v), bits = U.host_inputs(w)
    qkv = torch.zeros(w.B, w.n_alloc, 3, w.H, w.d, dtype=torch.bfloat16, device="cuda")
    for i, x in enumerate((q, k, v)):
        qkv[:, :, i] = U.dev(x).permute(0, 2, 1, 3)
    qv, kv, vv = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    rp, ci, _ = U.gpu_select(w, qv, kv)
    o_buf = torch.zeros(w.B, w.n_alloc, w.H, w.d, dtype=torch.bfloat16, device="cuda")
    o = o_buf.permute(0, 2, 1, 3)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = B.make_problem(qv, kv, vv, o, w.N, w.block)
    ws = torch.full((B.attn_workspace_bytes(p),), 0xFF, dtype=torch.uint8, device="cuda")
    B.block_sparse_attn_fwd(p, qv, kv, vv, rp, ci, o, None, st, workspace=ws)
    torch.cuda.synchronize()
    assert int(st) == 0
    U.check_attn_vs_oracle(w, *bits, rp, ci, o.contiguous(), None, U.sample_rows(w.R, w.Nb, 6))


def test_large_logits_need_rescaling():
    """Scores that grow along the key axis force the running maximum (and O) to be rescaled."""
    w = shrink(WORKLOADS["medium"], H=1, T=2, k=16)      # dense-ish: Nb = 16
    (q, k, v), _ = U.host_inputs(w)
    ramp = torch.linspace(0.2, 3.0, w.N)[None, None, :, None]
    k = (k.float() * ramp).bfloat16()
    q = (q.float() * 2.0).bfloat16()
    from paper_2606_23743_b200.workloads import bf16_bits
    bits = (bf16_bits(q), bf16_bits(k), bf16_bits(v))
    data = (U.dev(q), U.dev(k), U.dev(v))
    rp, ci, _ = U.gpu_select(w, data[0], data[1])
    o, lse, st = U.gpu_attn(w, *data, rp, ci)
    U.check_attn_vs_oracle(w, *bits, rp, ci, o, lse, list(range(w.R)))


def test_wait_that_runs_out_is_reported_and_the_context_survives():
    """Failure detection without faulting the GPU: one tile's K stream is withheld (test switch),
    the bounded waits expire, the kernel returns with SVA_DEV_TIMEOUT and the next call works."""
    import ctypes as C
    w = shrink(WORKLOADS["medium"], H=1, T=2, k=4)        # 16 rows -> 8 CTAs
    data, bits, rp, ci = _setup(w)
    L = B.lib()
    try:
        assert L.sva_debug_set_wait_limit(C.c_longlong(100_000_000)) == 0     # ~50 ms
        L.sva_debug_set_mode(16)
        o, lse, st = U.gpu_attn(w, *data, rp, ci)
        assert st & B.SVA_DEV_TIMEOUT
    finally:
        L.sva_debug_set_mode(0)
        L.sva_debug_set_wait_limit(C.c_longlong(0))
    o, lse, st = U.gpu_attn(w, *data, rp, ci)
    assert st == 0
    U.check_attn_vs_oracle(w, *bits, rp, ci, o, lse, list(range(w.R)))
