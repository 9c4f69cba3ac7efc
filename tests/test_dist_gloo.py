"""The N>1 plumbing on CPU: two gloo ranks shard sequences disjointly and the
timing reduction takes the max / the unit count the sum over ranks."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2603_08088_b200 import dist as tvd
    r, w, _ = tvd.init_from_env("gloo")
    mine = tvd.shard_sequences(7, r, w)
    tvd.barrier()
    t = tvd.max_over_ranks(10.0 + 5 * r)
    n = tvd.sum_over_ranks(len(mine))
    q.put((r, mine, t, n))


def test_two_rank_sharding_and_reductions():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][1] == [0, 2, 4, 6] and got[1][1] == [1, 3, 5]
    assert got[0][2] == got[1][2] == 15.0
    assert got[0][3] == got[1][3] == 7.0


def test_single_process_is_identity():
    from paper_2603_08088_b200 import dist as tvd
    assert tvd.shard_sequences(5, 0, 1) == [0, 1, 2, 3, 4]
    assert tvd.max_over_ranks(3.5) == 3.5 and tvd.sum_over_ranks(2) == 2.0
