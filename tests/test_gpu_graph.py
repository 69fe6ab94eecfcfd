"""The path inside a CUDA graph: the library allocates nothing and never synchronises, so routing, the V
transpose on a forked stream and attention can be captured once and replayed on new data in the same
buffers."""
import pytest
import torch

import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["large", "large_fp8"])
def test_capture_and_replay(name):
    w = shrink(WORKLOADS[name], H=2, T=3)
    (q, k, v), _ = U.host_inputs(w)
    (q2, k2, v2), _ = U.host_inputs(w, seed=99)
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    o = torch.zeros_like(vd)
    lse = torch.zeros(w.B, w.H, w.N, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pq = B.make_problem(qd, kd, None, None, w.N, w.block)
    if w.fp8:
        q8 = torch.zeros(qd.shape, dtype=torch.uint8, device="cuda"); k8 = torch.zeros_like(q8)
        qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device="cuda"); ks = torch.zeros_like(qs)
        p = B.make_problem(q8, k8, vd, o, w.N, w.block, 0.0, True)
    else:
        p = B.make_problem(qd, kd, vd, o, w.N, w.block)
    s = B.make_select(w.mode, w.k, w.tau)
    ws = torch.empty(B.select_workspace_bytes(p, s), dtype=torch.uint8, device="cuda")
    aws = torch.full((B.attn_workspace_bytes(p),), 0xFF, dtype=torch.uint8, device="cuda")
    rp = torch.zeros(w.R + 1, dtype=torch.int32, device="cuda")
    ci = torch.zeros(B.select_max_nnz(p, s), dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()

    def path():
        if w.fp8:
            B.quantize_qk_fp8(pq, qd, kd, q8, k8, qs, ks)
            B.block_select(p, s, q8, k8, rp, ci, ws, qs, ks)
            B.block_sparse_attn_fwd(p, q8, k8, vd, rp, ci, o, lse, status, qs, ks, workspace=aws)
        else:
            cur = torch.cuda.current_stream()
            side.wait_stream(cur)
            with torch.cuda.stream(side):
                B.attn_prepare_v(p, vd, aws)
            B.block_select(p, s, qd, kd, rp, ci, ws)
            cur.wait_stream(side)
            B.block_sparse_attn_fwd_prepared(p, qd, kd, rp, ci, o, lse, status, workspace=aws)

    def eager(a, b, c):
        qd.copy_(U.dev(a)); kd.copy_(U.dev(b)); vd.copy_(U.dev(c))
        path()
        torch.cuda.synchronize()
        return o.clone(), lse.clone(), rp.clone(), ci.clone()

    ref1 = eager(q, k, v)
    ref2 = eager(q2, k2, v2)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        path()
    for (a, b, c), ref in (((q, k, v), ref1), ((q2, k2, v2), ref2), ((q, k, v), ref1)):
        qd.copy_(U.dev(a)); kd.copy_(U.dev(b)); vd.copy_(U.dev(c))
        o.zero_(); lse.zero_(); rp.zero_(); ci.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(rp, ref[2]) and torch.equal(ci, ref[3])
        assert torch.equal(o, ref[0]) and torch.equal(lse, ref[1])
