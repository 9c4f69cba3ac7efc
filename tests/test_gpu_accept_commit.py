"""tree_accept and kv_commit on the GPU against the oracle: bit-exact argmax
tokens, gathered indices, accepted lengths / paths and committed KV bytes."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy, bf16_bits
from gpu_util import to_device, i32

pytestmark = pytest.mark.gpu


def gpu_accept(logits, tokens, retrieve, n_nodes, status_in=None):
    dev = "cuda"
    B, N, V = logits.shape
    P, Dp1 = retrieve.shape[1], retrieve.shape[2]
    z = lambda *s: torch.full(s, -9, dtype=torch.int32, device=dev)
    o = dict(argmax_tok=z(B, N), accept_len=z(B), best_path=z(B), accepted_nodes=z(B, Dp1), next_token=z(B),
             safe_idx=z(B, max(P, 1), Dp1), candidates=z(B, max(P, 1), Dp1))
    status = torch.zeros(B, dtype=torch.int32, device=dev) if status_in is None else status_in.to(dev)
    ws = torch.zeros(max(16, tv.tv_accept_workspace_bytes(B, N, V)), dtype=torch.uint8, device=dev)
    tv.tree_accept(logits.to(dev), tokens.to(dev), retrieve.to(dev), n_nodes.to(dev), o["argmax_tok"],
                   o["accept_len"], o["best_path"], o["accepted_nodes"], o["next_token"], ws, status,
                   safe_idx=o["safe_idx"], candidates=o["candidates"])
    torch.cuda.synchronize()
    res = {k: i32(v) for k, v in o.items()}
    res["status"] = i32(status)
    return res


def check_accept(logits, tokens, retrieve, n_nodes):
    got = gpu_accept(logits, tokens, retrieve, n_nodes)
    am = orc.argmax_rows(bf16_bits(logits), n_nodes.numpy())
    ref = orc.greedy_accept(retrieve.numpy(), tokens.numpy(), n_nodes.numpy(), am)
    assert np.array_equal(got["argmax_tok"], am), "argmax tokens differ"
    P = retrieve.shape[1]
    for k in ("accept_len", "best_path", "accepted_nodes", "next_token", "status"):
        assert np.array_equal(got[k], ref[k]), f"{k}: {got[k]} vs {ref[k]}"
    if P > 0:
        assert np.array_equal(got["safe_idx"], ref["safe_idx"]) and np.array_equal(got["candidates"], ref["candidates"])
    return got, ref


@pytest.mark.parametrize("ci,over", [(0, {}), (1, dict(V=32000)), (2, dict(B=3, V=128256)),
                                     (4, dict(B=4, V=153600, L=1)), (4, dict(B=5, V=8200, L=1)),
                                     (0, dict(B=3, V=1001)), (2, dict(B=2, V=7))])
def test_accept_parity(ci, over):
    cfg = CONFIGS[ci].scaled(S_lo=1, S_hi=8, Scap=32, L=1, **{k: v for k, v in over.items() if k != "L"})
    case = make_case(cfg, seed=1000 * ci + 3, ragged_nodes=(cfg.B > 1), with_cache=False)
    got, ref = check_accept(case["logits"], case["tokens"], case["retrieve"], case["n_nodes"])
    if cfg.plant != "none" and cfg.V > 5000:
        for b in range(cfg.B):
            if case["n_nodes"][b] == cfg.N:
                assert got["accept_len"][b] >= case["plant_depth"][b]


def test_argmax_ties_signed_zero_and_minus_infinity():
    B, N, V = 2, 6, 20000
    g = torch.Generator().manual_seed(5)
    logits = torch.randn(B, N, V, generator=g).to(torch.bfloat16)
    logits[0, 0, [19999, 8192, 8191]] = 9.0          # tie across chunk boundary: lowest index wins
    logits[0, 1, [3, 4, 5, 6]] = 9.0                 # tie inside one 16-byte vector
    logits[0, 2, :] = -0.0
    logits[0, 2, 12345] = 0.0                        # -0.0 == +0.0: index 0 wins
    logits[0, 3, :] = float("-inf")                  # all -inf: index 0
    logits[0, 4, :] = float("-inf")
    logits[0, 4, 16384] = -3.0                       # single finite entry at a chunk start
    logits[1, 0, :] = 1.0                            # all equal
    logits[1, 1, V - 1] = 50.0                       # very last element
    tokens = torch.zeros(B, N, dtype=torch.int32)
    retrieve = torch.full((B, 1, 2), -1, dtype=torch.int32)
    retrieve[:, 0, 0] = 0
    n = torch.tensor([6, 5], dtype=torch.int32)
    got, _ = check_accept(logits, tokens, retrieve, n)
    assert got["argmax_tok"][0, :5].tolist() == [8191, 3, 0, 0, 16384]
    assert got["argmax_tok"][1, 0] == 0 and got["argmax_tok"][1, 1] == V - 1 and got["argmax_tok"][1, 5] == -1


def test_accept_validity_guard_bad_indices_and_no_rows():
    V = 64
    logits = torch.full((3, 4, V), -1.0, dtype=torch.bfloat16)
    tokens = torch.tensor([[42, 5, 6, 7]] * 3, dtype=torch.int32)
    for b in range(3):
        logits[b, 0, 5] = 3.0     # am[0] = 5  -> accepts node 1
        logits[b, 1, 6] = 3.0     # am[1] = 6  -> accepts node 2
        logits[b, 2, 42] = 3.0    # am[2] = 42 == tokens[0]: the dummy slot must not match
        logits[b, 3, 1] = 3.0
    retrieve = torch.full((3, 2, 5), -1, dtype=torch.int32)
    retrieve[0, 0, :3] = torch.tensor([0, 1, 2])
    retrieve[1, 0, :3] = torch.tensor([0, 1, 2])
    retrieve[1, 1, :4] = torch.tensor([0, 1, 3, -5])      # -5: flagged, treated as padding
    retrieve[2, 1, :3] = torch.tensor([0, 1, 9])          # 9 >= n_nodes: flagged, remapped to 0
    n = torch.tensor([3, 4, 4], dtype=torch.int32)
    got, ref = check_accept(logits, tokens, retrieve, n)
    assert got["accept_len"].tolist() == [2, 2, 1]
    assert got["status"].tolist() == [0, orc.ST_BAD_INDEX, orc.ST_BAD_INDEX]
    assert got["next_token"][0] == 42
    # P = 0: nothing to accept, the root is committed, the bonus token is am[root]
    got, ref = check_accept(logits, tokens, torch.zeros(3, 0, 5, dtype=torch.int32), n)
    assert got["accept_len"].tolist() == [0, 0, 0] and got["next_token"].tolist() == [5, 5, 5]


def gpu_commit(case_np, nodes, A, S, status_in=None, guard=True):
    dev = "cuda"
    kc, vc = torch.from_numpy(case_np["k_cache"].view(np.int16)), torch.from_numpy(case_np["v_cache"].view(np.int16))
    kt, vt = torch.from_numpy(case_np["k_tree"].view(np.int16)), torch.from_numpy(case_np["v_tree"].view(np.int16))
    L, B = kc.shape[0], kc.shape[1]
    pad = 4096
    def guarded(t):
        flat = torch.full((t.numel() + 2 * pad,), 0x1234, dtype=torch.int16, device=dev)
        flat[pad:-pad] = t.reshape(-1).to(dev)
        return flat, flat[pad:-pad].view(t.shape)
    kflat, kcd = guarded(kc)
    vflat, vcd = guarded(vc)
    Sd = torch.from_numpy(S.astype(np.int32)).to(dev)
    st = torch.zeros(B, dtype=torch.int32, device=dev) if status_in is None else torch.from_numpy(status_in.astype(np.int32)).to(dev)
    tv.kv_commit(kcd.view(torch.bfloat16), vcd.view(torch.bfloat16), kt.to(dev).view(torch.bfloat16),
                 vt.to(dev).view(torch.bfloat16), torch.from_numpy(nodes.astype(np.int32)).to(dev),
                 torch.from_numpy(A.astype(np.int32)).to(dev), Sd, st)
    torch.cuda.synchronize()
    for flat in (kflat, vflat):
        assert (flat[:pad] == 0x1234).all() and (flat[-pad:] == 0x1234).all(), "commit wrote outside the cache"
    return (kcd.cpu().numpy().view(np.uint16), vcd.cpu().numpy().view(np.uint16), i32(Sd), i32(st))


@pytest.mark.parametrize("d,Hkv", [(64, 2), (128, 8), (128, 1), (256, 3)])
def test_commit_bytes_exact(d, Hkv):
    rng = np.random.default_rng(d + Hkv)
    L, B, Scap, N, Dp1 = 3, 5, 40, 17, 6
    u16 = lambda *s: rng.integers(0, 2 ** 16, size=s).astype(np.uint16)
    case_np = dict(k_cache=u16(L, B, Hkv, Scap, d), v_cache=u16(L, B, Hkv, Scap, d),
                   k_tree=u16(L, B, N, Hkv, d), v_tree=u16(L, B, N, Hkv, d))
    nodes = np.zeros((B, Dp1), dtype=np.int32)
    A = np.array([5, 0, 3, 2, 1], dtype=np.int32)
    for b in range(B):
        nodes[b, 1:A[b] + 1] = np.sort(rng.choice(np.arange(1, N), size=A[b], replace=False))
    S = np.array([0, 39, 35, 20, 38], dtype=np.int32)      # b=2: 35+4 = 39 fits; b=4: 38+2 = 40 fits exactly
    status_in = np.array([0, 0, 0, orc.ST_BAD_TREE, 0])
    kc, vc, S2, st = gpu_commit(case_np, nodes, A, S, status_in)
    rk, rv, rS, rst = orc.kv_commit(case_np["k_cache"], case_np["v_cache"], case_np["k_tree"], case_np["v_tree"],
                                    nodes, A, S, status_in)
    assert np.array_equal(kc, rk) and np.array_equal(vc, rv), "committed bytes differ"
    assert np.array_equal(S2, rS) and np.array_equal(st, rst)
    assert S2.tolist() == [6, 40, 39, 20, 40]
    # capacity overflow, bad node id, bad length: flagged and untouched
    S_bad = np.array([35, 0, 0, 0, 40], dtype=np.int32)
    nodes_bad = nodes.copy()
    nodes_bad[2, 1] = N
    A_bad = A.copy()
    A_bad[3] = Dp1
    kc, vc, S2, st = gpu_commit(case_np, nodes_bad, A_bad, S_bad)
    rk, rv, rS, rst = orc.kv_commit(case_np["k_cache"], case_np["v_cache"], case_np["k_tree"], case_np["v_tree"],
                                    nodes_bad, A_bad, S_bad)
    assert np.array_equal(kc, rk) and np.array_equal(vc, rv) and np.array_equal(S2, rS) and np.array_equal(st, rst)
    assert st.tolist() == [orc.ST_CAPACITY, 0, orc.ST_BAD_INDEX, orc.ST_BAD_INDEX, orc.ST_CAPACITY]


def test_many_sequences_accept_and_commit_at_the_row_limit():
    """tree_accept takes up to 65535 (sequence, node) rows: 512 sequences of 127 slots here, ragged, a small
    vocabulary; the commit behind it moves the accepted rows of all 512 sequences.  One row more is refused."""
    B, N, V = 512, 127, 301
    cfg = CONFIGS[0].scaled(B=B, N=N, D=5, V=V, S_lo=1, S_hi=8, Scap=32, L=1, Hq=2, Hkv=1, d=64, tree="uniform")
    case = make_case(cfg, seed=31337, ragged_nodes=True, with_cache=False)
    got, ref = check_accept(case["logits"], case["tokens"], case["retrieve"], case["n_nodes"])
    assert (ref["accept_len"] > 0).any()
    # commit of those paths: L = 2 layers, every byte
    rng = np.random.default_rng(5)
    L, Hkv, d, Scap, Dp1 = 2, 1, 64, 24, case["retrieve"].shape[2]
    u16 = lambda *s: rng.integers(0, 2 ** 16, size=s).astype(np.uint16)
    case_np = dict(k_cache=u16(L, B, Hkv, Scap, d), v_cache=u16(L, B, Hkv, Scap, d),
                   k_tree=u16(L, B, N, Hkv, d), v_tree=u16(L, B, N, Hkv, d))
    S = rng.integers(0, Scap - Dp1, size=B).astype(np.int32)
    kc, vc, S2, st = gpu_commit(case_np, ref["accepted_nodes"], ref["accept_len"], S, ref["status"])
    rk, rv, rS, rst = orc.kv_commit(case_np["k_cache"], case_np["v_cache"], case_np["k_tree"], case_np["v_tree"],
                                    ref["accepted_nodes"], ref["accept_len"], S, ref["status"])
    assert np.array_equal(kc, rk) and np.array_equal(vc, rv) and np.array_equal(S2, rS) and np.array_equal(st, rst)
    # 512 x 128 = 65536 rows: refused before anything is launched
    z = lambda *sh: torch.zeros(sh, dtype=torch.int32, device="cuda")
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_accept(torch.zeros(B, 128, 8, dtype=torch.bfloat16, device="cuda"), z(B, 128), z(B, 1, 2), z(B), z(B, 128), z(B),
                       z(B), z(B, 2), z(B), torch.zeros(1 << 20, dtype=torch.uint8, device="cuda"), z(B))


def test_node_scores_parity():
    """tree_node_scores against the oracle: bit-exact fp32 values of the gathered bf16 logits."""
    cfg = CONFIGS[4].scaled(S_lo=1, S_hi=8, Scap=32, L=1, B=6, V=153600)
    case = make_case(cfg, seed=77, ragged_nodes=True, with_cache=False)
    tokens = case["tokens"].clone()
    n = case["n_nodes"].numpy()
    bad = [b for b in range(cfg.B) if n[b] >= 2][:2]
    assert len(bad) == 2
    tokens[bad[0], int(n[bad[0]]) - 1] = cfg.V          # out of range: -inf and BAD_INDEX
    tokens[bad[1], 1] = -7
    tokens[bad[1], int(n[bad[1]]):] = -1                # padded slots are never looked at
    dev = "cuda"
    scores = torch.full((cfg.B, cfg.N), 5.0, dtype=torch.float32, device=dev)
    status = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    tv.tree_node_scores(case["logits"].to(dev), tokens.to(dev), case["parent"].to(dev), case["n_nodes"].to(dev),
                        scores, status)
    torch.cuda.synchronize()
    ref, ref_st = orc.node_scores(bf16_bits(case["logits"]), tokens.numpy(), case["parent"].numpy(),
                                  case["n_nodes"].numpy())
    assert np.array_equal(scores.cpu().numpy(), ref)
    assert np.array_equal(status.cpu().numpy(), ref_st)
    assert ref_st[bad[0]] == orc.ST_BAD_INDEX and np.isneginf(ref[bad[1], 1]) and (ref[:, 0] == 0).all()
