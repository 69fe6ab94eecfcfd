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
