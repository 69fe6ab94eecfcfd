"""The sequence-parallel wrapper on one GPU: a one-rank NCCL group, so that the CUDA `attend` callable and
the NCCL exchange calls run for real (the multi-rank exchange itself is covered on CPU with gloo)."""
import socket

import pytest
import torch
import torch.distributed as dist

import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200 import sequence_parallel as SP
from paper_2606_23743_b200.workloads import WORKLOADS, bf16_bits, shrink

pytestmark = pytest.mark.gpu


def test_one_rank_group_matches_the_direct_path_and_the_oracle():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        w = shrink(WORKLOADS["large"], H=2, T=2)
        (q, k, v), (qb, kb, vb) = U.host_inputs(w)
        qd, kd, vd = (U.dev(x)[:, :, :w.N].contiguous() for x in (q, k, v))
        sel = B.make_select(w.mode, w.k, w.tau)
        attend = SP.sparse_attend(sel, w.block)
        o = SP.sequence_parallel_attention(qd, kd, vd, SP.even_shards(w.N, 1), attend)
        torch.cuda.synchronize()
        assert int(attend.status.item()) == 0                 # what the kernels reported is not dropped
        rp, ci, _ = U.gpu_select(w, U.dev(q), U.dev(k))
        o_direct, _, st = U.gpu_attn(w, U.dev(q), U.dev(k), U.dev(v), rp, ci)
        assert st == 0 and torch.equal(o, o_direct[:, :, :w.N])
        U.check_attn_vs_oracle(w, qb, kb, vb, rp, ci, o, None, U.sample_rows(w.R, w.Nb, 6))
    finally:
        dist.destroy_process_group()
