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


def _split_worker(rank, world, port, q):
    """Context split on CPU: every rank attends (oracle) to its own key range, the partials travel through
    gather_partials, and the merged result must equal the attention over the whole prefix."""
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import numpy as np
    import torch
    from oracle import tree_verify_oracle as orc
    from paper_2603_08088_b200 import dist as tvd
    from workloads import CONFIGS, make_case, case_to_numpy
    r, w, _ = tvd.init_from_env("gloo")
    cfg = CONFIGS[0].scaled(B=2, S_lo=9, S_hi=41, Scap=48)
    c = case_to_numpy(make_case(cfg, seed=5, ragged_nodes=True))          # same seeded case on every rank
    S = c["prefix_len"].astype(np.int64)
    vis = orc.build_mask(c["parent"], c["n_nodes"], cfg.N - 1, 1, emit_paths=False)["dense"][:, 0]
    scale = cfg.d ** -0.5
    lo, hi = tvd.split_prefix(S, r, w)
    kc, vc = np.zeros_like(c["k_cache"][0]), np.zeros_like(c["v_cache"][0])
    for b in range(cfg.B):
        kc[b, :, :hi[b] - lo[b]] = c["k_cache"][0][b, :, lo[b]:hi[b]]
        vc[b, :, :hi[b] - lo[b]] = c["v_cache"][0][b, :, lo[b]:hi[b]]
    owns_tree = r == w - 1
    o, l = orc.tree_attention(c["q"][0], kc, vc, c["k_tree"][0], c["v_tree"][0], hi - lo, c["n_nodes"],
                              vis if owns_tree else np.zeros_like(vis), scale)
    o_parts, l_parts = tvd.gather_partials(torch.from_numpy(o), torch.from_numpy(l))
    out, lse = orc.merge_partials(o_parts.numpy(), l_parts.numpy())
    full, full_lse = orc.tree_attention(c["q"][0], c["k_cache"][0], c["v_cache"][0], c["k_tree"][0], c["v_tree"][0],
                                        S, c["n_nodes"], vis, scale)
    fin = np.isfinite(full_lse)
    q.put((r, tuple(o_parts.shape), float(np.abs(out - full).max()), float(np.abs(lse[fin] - full_lse[fin]).max()),
           bool(np.array_equal(np.isneginf(lse), np.isneginf(full_lse))), [int(x) for x in lo], [int(x) for x in hi]))


def test_two_rank_context_split_matches_attention_over_the_whole_prefix():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_split_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r, shape, err_o, err_l, same_inf, lo, hi in got:
        assert shape[0] == 2 and err_o < 1e-12 and err_l < 1e-12 and same_inf
    assert got[0][5] == [0, 0] and got[0][6] == got[1][5]          # ranges tile the prefix without a gap


def test_split_prefix_tiles_the_prefix():
    import torch
    from paper_2603_08088_b200 import dist as tvd
    S = torch.tensor([0, 1, 7, 4096, 32768 + 5])
    for world in (1, 2, 3, 8):
        prev = torch.zeros_like(S)
        for r in range(world):
            lo, hi = tvd.split_prefix(S, r, world)
            assert torch.equal(lo, prev) and bool((hi >= lo).all())
            prev = hi
        assert torch.equal(prev, S)
