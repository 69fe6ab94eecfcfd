"""World-size-2 gloo run of the replica plumbing the bench uses at N > 1."""
import os
import socket

import torch.multiprocessing as mp


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2606_23743_b200 import dist as D
    r, lr, w = D.init("gloo")
    D.barrier()
    mx = D.max_over_ranks(10.0 + rank)
    sm = D.sum_over_ranks(100.0 * (rank + 1))
    seed = D.rank_seed(23743003, r)
    D.finalize()
    q.put((r, w, mx, sm, seed))


def test_two_rank_replicas_gloo():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    out = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [o[0] for o in out] == [0, 1] and all(o[1] == 2 for o in out)
    assert all(o[2] == 11.0 for o in out)          # max over ranks
    assert all(o[3] == 300.0 for o in out)         # whole-job aggregate
    assert out[0][4] != out[1][4]                  # different batch sample per replica


def test_single_process_is_identity():
    from paper_2606_23743_b200 import dist as D
    assert D.max_over_ranks(3.5) == 3.5 and D.sum_over_ranks(2.0) == 2.0


# ------------------------------------------------------------------ sequence-parallel exchange (world 2 and 3, gloo)
def _sp_worker(rank, world, port, q, N, H, B_=2):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch
    from paper_2606_23743_b200 import dist as D
    from paper_2606_23743_b200 import sequence_parallel as SP
    D.init("gloo")
    g = torch.Generator().manual_seed(5)
    d = 8
    full = [torch.randn(B_, H, N, d, generator=g) for _ in range(3)]          # the same on every rank
    sizes = SP.even_shards(N, world)
    lo, hi = SP.shard_bounds(sizes)[rank]
    hg = H // world
    mine = [x[:, :, lo:hi].contiguous() for x in full]
    # exchange: my heads of all tokens
    qh = SP.seq_to_head_shard(mine[0], sizes)
    ok_fwd = torch.equal(qh, full[0][:, rank * hg:(rank + 1) * hg])
    # and back
    ok_back = torch.equal(SP.head_to_seq_shard(qh, sizes), mine[0])

    # whole thing with a plain dense attention as the per-rank step, against the unsharded result
    def attend(q_, k_, v_):
        return torch.softmax(q_ @ k_.transpose(-1, -2) / d ** 0.5, dim=-1) @ v_
    o = SP.sequence_parallel_attention(mine[0], mine[1], mine[2], sizes, attend)
    ref = attend(*full)[:, :, lo:hi]
    err = float((o - ref).abs().max()) if o.numel() else 0.0
    # wrong arguments raise before any communication
    bad = 0
    try:
        SP.seq_to_head_shard(mine[0][:, :H - 1], sizes)
    except ValueError:
        bad += 1
    try:
        SP.seq_to_head_shard(mine[0], sizes[:-1])
    except ValueError:
        bad += 1
    D.barrier()
    D.finalize()
    q.put((rank, ok_fwd, ok_back, tuple(o.shape), err, bad))


def _run_sp(world, N, H, B_=2):
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_sp_worker, args=(r, world, port, q, N, H, B_)) for r in range(world)]
    for p in ps:
        p.start()
    out = sorted(q.get(timeout=180) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    return out


def test_sequence_parallel_exchange_two_ranks_even():
    out = _run_sp(2, 64, 4)
    for rank, ok_fwd, ok_back, shape, err, bad in out:
        assert ok_fwd and ok_back and bad == 2
        assert shape == (2, 4, 32, 8) and err < 1e-5


def test_sequence_parallel_exchange_three_ranks_ragged():
    """N = 50 over 3 ranks: shards of 17, 17, 16 tokens; 6 heads -> 2 per rank."""
    out = _run_sp(3, 50, 6)
    assert [o[3][2] for o in out] == [17, 17, 16]
    for rank, ok_fwd, ok_back, shape, err, bad in out:
        assert ok_fwd and ok_back and bad == 2 and err < 1e-5


def test_sequence_parallel_exchange_one_batch_entry_ragged():
    """B = 1 takes the forms of the two exchanges that skip a staging copy (the head groups of a contiguous
    one-entry tensor already lie one behind the other): same checks, 3 ranks, ragged shards."""
    out = _run_sp(3, 50, 6, 1)
    assert [o[3] for o in out] == [(1, 6, 17, 8), (1, 6, 17, 8), (1, 6, 16, 8)]
    for rank, ok_fwd, ok_back, shape, err, bad in out:
        assert ok_fwd and ok_back and bad == 2 and err < 1e-5


def test_shard_helpers():
    from paper_2606_23743_b200 import sequence_parallel as SP
    assert SP.even_shards(10, 4) == [3, 3, 3, 1] and SP.even_shards(4, 8) == [1, 1, 1, 1, 0, 0, 0, 0]
    assert SP.shard_bounds([3, 3, 3, 1]) == [(0, 3), (3, 6), (6, 9), (9, 10)]
    assert sum(SP.even_shards(32760, 4)) == 32760
