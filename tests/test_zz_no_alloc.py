"""The routing entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not theirs to call (a plugin that only
gets input and output buffers, a step inside a region that must not touch the allocator), so
sva_block_select_noalloc takes its scratch from a 16 MiB device array built into the library.
It runs the same kernels as sva_block_select, so its CSR and scores must be identical -- on a
first call and again on a second call that finds the previous call's bytes in the scratch.
This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes as C

import pytest
import torch

import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu


def _both(w, q, k):
    """(row_ptr, col_idx, scores) from the allocating entry point and from the no-alloc one."""
    rp_a, ci_a, sc_a = U.gpu_select(w, q, k, want_scores=True)
    p = B.make_problem(q, k, None, None, w.N, w.block)
    s = B.make_select(w.mode, w.k, w.tau, w.win_t, w.win_s, w.blocks_per_frame if w.win_t >= 0 else 0)
    assert B.select_workspace_bytes(p, s) <= B.NOALLOC_SCRATCH_BYTES
    rp_b = torch.full((w.R + 1,), -7, dtype=torch.int32, device="cuda")
    ci_b = torch.full((B.select_max_nnz(p, s),), -7, dtype=torch.int32, device="cuda")
    sc_b = torch.empty_like(sc_a)
    B.block_select_noalloc(p, s, q, k, rp_b, ci_b, block_scores=sc_b)
    torch.cuda.synchronize()
    return (rp_a, ci_a, sc_a), (rp_b, ci_b[: int(rp_b[-1])], sc_b)


def test_noalloc_matches_allocating_entry_point_twice_in_a_row():
    # first call: mass rule with ragged rows (staging, scan and compaction all use the scratch)
    w1 = shrink(WORKLOADS["large_ragged"], H=4, T=8)
    (q1, k1, _), _ = U.host_inputs(w1)
    a, b = _both(w1, U.dev(q1), U.dev(k1))
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    # second call, different shape and rule, straight after: stale scratch contents must not matter
    w2 = shrink(WORKLOADS["xl"], B=1, H=2, T=5, k=5)          # forced window larger than k
    (q2, k2, _), _ = U.host_inputs(w2)
    a, b = _both(w2, U.dev(q2), U.dev(k2))
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    # and the first problem again gives the first answer again
    a2, b2 = _both(w1, U.dev(q1), U.dev(k1))
    assert torch.equal(a2[1], b2[1])


def test_noalloc_rejects_problems_beyond_its_scratch():
    w = WORKLOADS["xl"]                                        # pooled means alone are 24 MB
    # describe the full-size problem without allocating it: the size check is host-side and
    # comes before any launch, so the tensors are never read
    small = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    p = B.Problem()
    p.B, p.H, p.N, p.d, p.block = w.B, w.H, w.N, w.d, w.block
    for f in ("q_stride", "k_stride", "v_stride", "o_stride"):
        setattr(p, f, (C.c_int64 * 3)(w.H * w.n_alloc * w.d, w.n_alloc * w.d, w.d))
    s = B.make_select(w.mode, w.k, w.tau, w.win_t, w.win_s, w.blocks_per_frame)
    assert B.select_workspace_bytes(p, s) > B.NOALLOC_SCRATCH_BYTES
    with pytest.raises(B.SvaError) as e:
        B.block_select_noalloc(p, s, small, small, small, small)
    assert e.value.status == 6 and "scratch" in str(e.value)
