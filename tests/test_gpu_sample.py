"""tree_accept_sample on the GPU against the oracle.  The kernel decides in fp32 and the oracle in fp64, so
accept decisions, node lists and status are compared bit-exactly wherever the oracle's own decisions do not
hinge on the last bits of a uniform, and the drawn token is checked as a valid inversion of the oracle's
cumulative distribution (see check())."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import bf16_bits, random_parent_tree, topk_expansion_tree

pytestmark = pytest.mark.gpu


def make_inputs(seed, B, N, D, V, tree="uniform", hot=(5.0, 9.0), ragged=False):
    rng = np.random.default_rng(seed)
    parent = np.zeros((B, N), dtype=np.int32)
    for b in range(B):
        parent[b] = random_parent_tree(N, D, rng) if tree == "uniform" else topk_expansion_tree(N, D, 8, rng)
    n = np.full(B, N, dtype=np.int32)
    if ragged:
        n[1:] = rng.integers(1, N + 1, size=B - 1)
    logits = rng.standard_normal((B, N, V)).astype(np.float32)
    tokens = rng.integers(0, V, size=(B, N)).astype(np.int32)
    for b in range(B):
        for k in range(1, N):
            if rng.random() < 0.15 and k > 1:
                tokens[b, k] = tokens[b, k - 1]            # sibling duplicates now and then
            logits[b, parent[b, k], tokens[b, k]] = rng.uniform(*hot)    # give the proposals real probability
    lt = torch.from_numpy(logits).to(torch.bfloat16)
    u_node = rng.random((B, N)).astype(np.float32)
    u_bonus = rng.random(B).astype(np.float32)
    return lt, tokens, parent, n, u_node, u_bonus


def run_gpu(lt, tokens, parent, n, u_node, u_bonus, T, Dp1, status_in=None):
    dev = "cuda"
    B, N, V = lt.shape
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev)
    alen = torch.full((B,), -9, dtype=torch.int32, device=dev)
    nodes = torch.full((B, Dp1), -9, dtype=torch.int32, device=dev)
    nxt = torch.full((B,), -9, dtype=torch.int32, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev) if status_in is None else i32(status_in)
    ws = torch.zeros(max(16, tv.tv_sample_workspace_bytes(B, N, V)), dtype=torch.uint8, device=dev)
    tv.tree_accept_sample(lt.to(dev), i32(tokens), i32(parent), i32(n), f32(u_node), f32(u_bonus), T, alen, nodes, nxt,
                          ws, status)
    torch.cuda.synchronize()
    return {"accept_len": alen.cpu().numpy(), "accepted_nodes": nodes.cpu().numpy(), "next_token": nxt.cpu().numpy(),
            "status": status.cpu().numpy()}


def check(lt, tokens, parent, n, u_node, u_bonus, T, Dp1, min_fraction=0.8):
    """Accept decisions, node lists and status must equal the oracle's wherever the oracle's own decisions do
    not move when every u_node is shifted by +-2e-5 (relative).  The drawn token must be a valid inversion:
    the target u_bonus * (remaining mass) lies in the token's interval of the fp64 cumulative sum, give or take
    2e-5 of the total (an fp32 cumulative sum over 10^5 entries cannot promise more), and the token has mass."""
    bits = bf16_bits(lt)
    got = run_gpu(lt, tokens, parent, n, u_node, u_bonus, T, Dp1)
    refs = [orc.stochastic_accept(bits, tokens, parent, n, np.clip(u_node.astype(np.float64) * f, 0, 1 - 1e-12),
                                  u_bonus.astype(np.float64), T, Dp1)
            for f in (1.0, 1.0 - 2e-5, 1.0 + 2e-5)]
    B, N, V = lt.shape
    compared = 0
    for b in range(B):
        stable = all(np.array_equal(r[key][b], refs[0][key][b]) for r in refs[1:] for key in ("accept_len", "accepted_nodes"))
        if not stable:
            continue
        compared += 1
        for key in ("accept_len", "accepted_nodes", "status"):
            assert np.array_equal(got[key][b], refs[0][key][b]), f"sequence {b}: {key}: {got[key][b]} vs {refs[0][key][b]}"
        nb = int(min(max(n[b], 0), N))
        if nb == 0:
            assert got["next_token"][b] == -1
            continue
        a = int(got["accept_len"][b])
        c = int(got["accepted_nodes"][b, a])
        rejected = set()
        if a < Dp1 - 1:      # every child of the last node was tried and failed
            rejected = {int(tokens[b, k]) for k in range(c + 1, nb) if parent[b, k] == c and 0 <= tokens[b, k] < V}
        row = orc.decode_bf16(bits[b, c]).astype(np.float64) / T
        kept = np.exp(row - row.max())
        kept[list(rejected)] = 0.0
        cum = np.cumsum(kept)
        target, tol = float(u_bonus[b]) * cum[-1], 2e-5 * cum[-1]
        v = int(got["next_token"][b])
        assert 0 <= v < V and kept[v] > 0.0, f"sequence {b}: token {v} has no mass"
        lo = cum[v - 1] if v > 0 else 0.0
        assert lo - tol <= target <= cum[v] + tol, f"sequence {b}: token {v} covers [{lo}, {cum[v]}], target {target}"
        if abs(target - lo) > tol and abs(target - cum[v]) > tol:
            assert v == refs[0]["next_token"][b]
    assert compared >= min_fraction * B, f"only {compared} of {B} sequences had decisions clear of rounding"
    return got, refs[0]


CASES = [
    # seed, B, N, D, V, tree, T
    (1, 6, 15, 4, 1024, "uniform", 1.0),
    (2, 5, 60, 6, 32000, "topk", 0.7),
    (3, 3, 64, 7, 128256, "topk", 1.0),
    (4, 6, 31, 5, 1001, "uniform", 1.3),          # V not a multiple of 8: scalar loads
    (5, 4, 128, 8, 8192, "topk", 0.5),
    (6, 2, 256, 8, 4096, "uniform", 2.0),
]


@pytest.mark.parametrize("seed,B,N,D,V,tree,T", CASES)
def test_sample_accept_parity(seed, B, N, D, V, tree, T):
    lt, tokens, parent, n, u_node, u_bonus = make_inputs(seed, B, N, D, V, tree, ragged=(B > 2))
    got, ref = check(lt, tokens, parent, n, u_node, u_bonus, T, D + 1)
    # every accepted list is a path from the root through parent links
    for b in range(B):
        a = int(got["accept_len"][b])
        path = got["accepted_nodes"][b, :a + 1].tolist()
        assert path[0] == 0 and all(parent[b, path[j]] == path[j - 1] for j in range(1, a + 1))
        assert (got["accepted_nodes"][b, a + 1:] == 0).all()
        assert 0 <= got["next_token"][b] < V


def test_sample_accept_exercises_both_outcomes_and_depth_cap():
    lt, tokens, parent, n, u_node, u_bonus = make_inputs(7, 16, 40, 6, 2048, "topk", hot=(6.0, 10.0))
    got, ref = check(lt, tokens, parent, n, u_node, u_bonus, 1.0, 7)
    assert got["accept_len"].max() >= 2 and got["accept_len"].min() == 0
    # Dp1 = 2: at most one accepted node, then the token is drawn at that node
    got2, _ = check(lt, tokens, parent, n, u_node, u_bonus, 1.0, 2)
    assert got2["accept_len"].max() == 1
    assert np.array_equal(got2["accepted_nodes"][:, 1] > 0, got["accept_len"] >= 1)


def test_sample_accept_low_temperature_is_the_greedy_rule():
    lt, tokens, parent, n, u_node, u_bonus = make_inputs(8, 5, 30, 5, 4096, "uniform", hot=(7.0, 7.0))
    # one clear maximum per row, carried by some child
    rng = np.random.default_rng(8)
    l = lt.float().numpy()
    for b in range(5):
        for i in range(30):
            kids = [k for k in range(i + 1, 30) if parent[b, k] == i]
            tok = tokens[b, kids[rng.integers(len(kids))]] if kids and rng.random() < 0.7 else rng.integers(4096)
            l[b, i, tok] = 12.0
    lt = torch.from_numpy(l).to(torch.bfloat16)
    got, _ = check(lt, tokens, parent, n, u_node, u_bonus, 0.02, 6, min_fraction=1.0)
    am = orc.argmax_rows(bf16_bits(lt), n)
    for b in range(5):
        c, path = 0, [0]
        while len(path) < 6:
            nxt = [k for k in range(c + 1, 30) if parent[b, k] == c and tokens[b, k] == am[b, c]]
            if not nxt:
                break
            c = nxt[0]
            path.append(c)
        assert got["accept_len"][b] == len(path) - 1 and got["accepted_nodes"][b, :len(path)].tolist() == path
        assert got["next_token"][b] == am[b, c]      # all the mass sits on the maximum


def test_sample_accept_flags_and_edges():
    lt, tokens, parent, n, u_node, u_bonus = make_inputs(9, 4, 12, 3, 512, "uniform")
    tokens[1, 3] = 512                      # outside the vocabulary
    tokens[2, 5] = -1
    n[3] = 0                                # no nodes at all
    got, ref = check(lt, tokens, parent, n, u_node, u_bonus, 1.0, 4, min_fraction=0.7)
    assert got["status"].tolist() == [0, tv.TV_ST_BAD_INDEX, tv.TV_ST_BAD_INDEX, 0]
    assert got["next_token"][3] == -1 and got["accept_len"][3] == 0
    # u = 0 accepts the first child that has any mass; u just below 1 rejects every child
    z = np.zeros_like(u_node)
    g0 = run_gpu(lt, tokens, parent, n, z, u_bonus, 1.0, 4)
    r0 = orc.stochastic_accept(bf16_bits(lt), tokens, parent, n, z, u_bonus, 1.0, 4)
    assert np.array_equal(g0["accepted_nodes"], r0["accepted_nodes"]) and g0["accept_len"][0] >= 1
    one = np.full_like(u_node, np.float32(1.0 - 2.0 ** -24))
    g1 = run_gpu(lt, tokens, parent, n, one, u_bonus, 1.0, 4)
    assert (g1["accept_len"] == 0).all()
    with pytest.raises(tv.TreeVerifyError):
        run_gpu(lt, tokens, parent, n, u_node, u_bonus, 0.0, 4)
