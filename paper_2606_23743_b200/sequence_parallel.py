"""Sequence-parallel wrapper around the single-GPU path (the paper runs one of its models with sequence
parallelism over 4 GPUs and names no collective; this is the head-exchange form).

Every rank holds all H heads of its own contiguous shard of the token sequence.  Attention needs whole
sequences, and its heads are independent, so one all-to-all turns "all heads of my tokens" into "my
H/G heads of all tokens", the unchanged single-GPU routing + attention runs on those heads, and the
inverse all-to-all brings every rank the output rows of its own tokens:

    [B, H, n_r, d] on rank r  --all-to-all-->  [B, H/G, N, d]  --route + attend-->  [B, H/G, N, d]
                              --all-to-all-->  [B, H, n_r, d]

Per tensor and direction a rank sends B*(H/G)*n_r*d elements to each peer.  Shards may differ in length
(`shard_sizes`, the same list on every rank); H must be a multiple of the group size.  The exchange is
`torch.distributed.all_to_all_single` with split sizes (NCCL on GPUs, gloo on CPU for the tests); nothing here
computes.
"""
from __future__ import annotations

from typing import Callable, Sequence

import torch
import torch.distributed as dist


def shard_bounds(shard_sizes: Sequence[int]):
    """[(lo, hi)] of every rank's token range in the full sequence."""
    out, lo = [], 0
    for n in shard_sizes:
        if n < 0:
            raise ValueError("negative shard size")
        out.append((lo, lo + n))
        lo += n
    return out


def even_shards(N: int, world: int):
    """ceil(N/world) tokens per rank, the tail shorter (possibly empty)."""
    per = -(-N // world)
    return [max(0, min(per, N - r * per)) for r in range(world)]


def _check(x: torch.Tensor, world: int, shard_sizes: Sequence[int]):
    if x.dim() != 4:
        raise ValueError("tensors are [B, H, n, d]")
    if len(shard_sizes) != world:
        raise ValueError(f"{len(shard_sizes)} shard sizes for a group of {world}")


def _exchange(send, recv_counts, group, src=None):
    """One all-to-all of flat chunks: send[g] goes to rank g, the result's entry s came from rank s.
    (The single-buffer form with split sizes: both the NCCL and the gloo backend have it.)
    `src`: the chunks as one flat buffer, when the caller's tensor already is that (no staging copy)."""
    if src is None:
        src = torch.cat(send)
    dst = src.new_empty(sum(recv_counts))
    dist.all_to_all_single(dst, src, output_split_sizes=list(recv_counts),
                           input_split_sizes=[t.numel() for t in send], group=group)
    return dst, list(torch.split(dst, list(recv_counts)))


def seq_to_head_shard(x_local: torch.Tensor, shard_sizes: Sequence[int], group=None) -> torch.Tensor:
    """[B, H, n_rank, d] (all heads, my tokens) -> [B, H/G, N, d] (my heads, all tokens)."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    _check(x_local, world, shard_sizes)
    Bq, H, n, d = x_local.shape
    if H % world:
        raise ValueError(f"H = {H} is not a multiple of the group size {world}")
    if n != shard_sizes[rank]:
        raise ValueError(f"rank {rank} holds {n} tokens, shard_sizes says {shard_sizes[rank]}")
    hg = H // world
    send = [x_local[:, g * hg:(g + 1) * hg].reshape(-1) for g in range(world)]
    # (one batch entry, contiguous: the head groups lie one behind the other already)
    flat = x_local.reshape(-1) if Bq == 1 and x_local.is_contiguous() else None
    _, recv = _exchange(send, [Bq * hg * shard_sizes[s] * d for s in range(world)], group, flat)
    return torch.cat([r.view(Bq, hg, shard_sizes[s], d) for s, r in enumerate(recv)], dim=2)


def head_to_seq_shard(x_heads: torch.Tensor, shard_sizes: Sequence[int], group=None) -> torch.Tensor:
    """[B, H/G, N, d] (my heads, all tokens) -> [B, H, n_rank, d] (all heads, my tokens)."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    _check(x_heads, world, shard_sizes)
    Bq, hg, N, d = x_heads.shape
    if N != sum(shard_sizes):
        raise ValueError(f"{N} tokens, shard sizes add up to {sum(shard_sizes)}")
    send = [x_heads[:, :, lo:hi].reshape(-1) for lo, hi in shard_bounds(shard_sizes)]
    dst, recv = _exchange(send, [Bq * hg * shard_sizes[rank] * d] * world, group)
    if Bq == 1:                                  # the received head groups already lie in head order
        return dst.view(1, hg * world, shard_sizes[rank], d)
    return torch.cat([r.view(Bq, hg, shard_sizes[rank], d) for r in recv], dim=1)


def sequence_parallel_attention(q_local: torch.Tensor, k_local: torch.Tensor, v_local: torch.Tensor,
                                shard_sizes: Sequence[int],
                                attend: Callable[[torch.Tensor, torch.Tensor, torch.Tensor], torch.Tensor],
                                group=None) -> torch.Tensor:
    """Exchange, run `attend(q, k, v) -> o` on this rank's heads over the full sequence, exchange back.
    `attend` is the single-GPU path (see `sparse_attend`); it sees [B, H/G, N, d] tensors."""
    q, k, v = (seq_to_head_shard(x, shard_sizes, group) for x in (q_local, k_local, v_local))
    return head_to_seq_shard(attend(q, k, v), shard_sizes, group)


def sparse_attend(select, block: int = 128, status=None):
    """The library's routing + block-sparse attention as an `attend` callable for CUDA bf16 tensors
    (select: a `binding.Select`).  Buffers are allocated per call; a serving loop would keep them.
    `status`: optional caller-owned device int32[1] that the kernels OR their SVA_DEV_* bits into (zero it
    first); without one the callable allocates its own.  Either way the word the last call used is
    `attend.status` -- read it after a synchronisation; a non-zero value means the output is not valid."""
    from . import binding as B

    def attend(q, k, v):
        if not q.is_cuda:
            raise RuntimeError("sparse_attend runs the CUDA library: tensors must be on a GPU (there is no CPU path)")
        N = q.shape[2]
        o = torch.empty_like(v)
        p = B.make_problem(q, k, v, o, N, block)
        R = q.shape[0] * q.shape[1] * (-(-N // block))
        ws = torch.empty(max(B.select_workspace_bytes(p, select), 256), dtype=torch.uint8, device=q.device)
        row_ptr = torch.zeros(R + 1, dtype=torch.int32, device=q.device)
        col_idx = torch.zeros(max(B.select_max_nnz(p, select), 1), dtype=torch.int32, device=q.device)
        st = status if status is not None else torch.zeros(1, dtype=torch.int32, device=q.device)
        attend.status = st
        aws = torch.empty(max(B.attn_workspace_bytes(p), 256), dtype=torch.uint8, device=q.device)
        B.block_select(p, select, q, k, row_ptr, col_idx, ws)
        B.block_sparse_attn_fwd(p, q, k, v, row_ptr, col_idx, o, None, st, workspace=aws)
        return o

    attend.status = status
    return attend
