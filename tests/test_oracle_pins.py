"""Pins for the CPU oracle: each part is checked against something other than
itself - a hand-worked fixture, brute force written differently, closed forms,
special trees that reduce to textbook routines, and library routines."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import tree_verify_oracle as orc
from workloads import (chain_tree, star_tree, random_parent_tree, topk_expansion_tree,
                       leaf_paths, bf16_bits, randn_bf16)

GOLD = os.path.join(os.path.dirname(__file__), "golden", "tree6_hand_worked.json")


def _bf16(x):
    return bf16_bits(torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def _anc_set_by_walk(parent, i):
    """Independent of the oracle: climb parent pointers from i to the root."""
    s = set()
    while i >= 0:
        s.add(int(i))
        i = int(parent[i])
    return s


def _random_trees(seed, count=12):
    rng = np.random.default_rng(seed)
    trees = []
    for t in range(count):
        if t % 2 == 0:
            N = int(rng.integers(2, 70))
            D = int(rng.integers(1, min(N - 1, 9) + 1))
            trees.append((random_parent_tree(N, D, rng), D))
        else:
            D = int(rng.integers(2, 9))
            k = 4 + t % 5
            N = int(rng.integers(D + 1, min(130, k + (D - 1) * k * k) + 1))
            trees.append((topk_expansion_tree(N, D, k, rng), D))
    return trees


# ------------------------------------------------------------------ mask ----
def test_golden_hand_worked_mask_and_accept():
    g = json.load(open(GOLD))
    parent = np.array([g["parent"]], dtype=np.int32)
    n = np.array([6], dtype=np.int32)
    mk = orc.build_mask(parent, n, Dcap=2, Pcap=4)
    assert mk["status"][0] == 0
    assert mk["dense"][0, 0].tolist() == g["dense_mask"]
    assert mk["anc_bits"][0, :, 0].tolist() == g["anc_bits"]
    assert mk["depth"][0].tolist() == g["depth"]
    assert mk["anc_table"][0].tolist() == g["anc_table"]
    assert mk["n_paths"][0] == 3
    assert mk["retrieve"][0, :3].tolist() == g["retrieve"]
    assert (mk["retrieve"][0, 3] == -1).all()
    am = np.array([g["teacher_argmax"]], dtype=np.int32)
    acc = orc.greedy_accept(mk["retrieve"], np.array([g["tokens"]], dtype=np.int32), n, am)
    assert acc["accept_len"][0] == g["accept_len"]
    assert acc["best_path"][0] == g["best_path"]
    assert acc["accepted_nodes"][0].tolist() == g["accepted_nodes"]
    assert acc["next_token"][0] == g["next_token"]
    # accepted length of every candidate row on its own: the rule applied to a one-row table
    toks = np.array([g["tokens"]], dtype=np.int32)
    per_path = [int(orc.greedy_accept(mk["retrieve"][:, p:p + 1], toks, n, am)["accept_len"][0]) for p in range(3)]
    assert per_path == g["per_path_accept"]
    assert max(per_path) == g["accept_len"] and per_path.index(max(per_path)) == g["best_path"]


def test_mask_equals_parent_walk_and_invariants():
    for parent, D in _random_trees(1):
        N = len(parent)
        mk = orc.build_mask(parent[None], np.array([N]), Dcap=D, Pcap=N)
        assert mk["status"][0] == 0
        vis = mk["dense"][0, 0]
        depth = mk["depth"][0]
        for i in range(N):
            anc = _anc_set_by_walk(parent, i)
            assert set(np.flatnonzero(vis[i]).tolist()) == anc
            assert vis[i, i] == 1 and vis[i, 0] == 1
            assert vis[i].sum() == depth[i] + 1 == len(anc)
            for j in np.flatnonzero(vis[i]):
                if j > 0:
                    assert vis[i, parent[j]] == 1          # ancestor-closed
            bits = 0
            for w in range(mk["anc_bits"].shape[2]):
                bits |= int(mk["anc_bits"][0, i, w]) << (32 * w)
            assert bits == sum(1 << j for j in anc)
        assert (np.triu(vis, 1) == 0).all()                # lower triangular
        # siblings differ only in their own bits
        for i in range(1, N):
            for j in range(i + 1, N):
                if parent[i] == parent[j]:
                    diff = np.flatnonzero(vis[i] != vis[j])
                    assert diff.tolist() == [i, j]


def test_mask_special_trees():
    N = 17
    mk = orc.build_mask(chain_tree(N)[None], np.array([N]), Dcap=N - 1, Pcap=2)
    assert (mk["dense"][0, 0] == np.tril(np.ones((N, N), dtype=np.uint8))).all()   # causal mask
    assert mk["n_paths"][0] == 1 and mk["retrieve"][0, 0].tolist() == list(range(N))
    mk = orc.build_mask(star_tree(N)[None], np.array([N]), Dcap=1, Pcap=N)
    want = np.eye(N, dtype=np.uint8)
    want[:, 0] = 1
    assert (mk["dense"][0, 0] == want).all()
    assert mk["n_paths"][0] == N - 1


def test_ancestor_table_is_l_fold_parent_and_in_range():
    for parent, D in _random_trees(2):
        N = len(parent)
        mk = orc.build_mask(parent[None], np.array([N]), Dcap=D + 2, Pcap=N)
        A = mk["anc_table"][0]
        assert A.min() >= 0 and A.max() < N
        for i in range(N):
            cur = i
            for l in range(D + 3):
                assert A[l, i] == cur
                cur = max(int(parent[cur]), 0)
            assert A[mk["depth"][0, i], i] == 0


def test_retrieve_rows_match_independent_leaf_walk():
    for parent, D in _random_trees(3):
        N = len(parent)
        mk = orc.build_mask(parent[None], np.array([N]), Dcap=D, Pcap=N)
        rows = leaf_paths(parent)
        assert mk["n_paths"][0] == len(rows)
        for p, r in enumerate(rows):
            assert mk["retrieve"][0, p, :len(r)].tolist() == r
            assert (mk["retrieve"][0, p, len(r):] == -1).all()
        # truncation keeps the first rows and raises the non-fatal bit
        if len(rows) > 1:
            mk2 = orc.build_mask(parent[None], np.array([N]), Dcap=D, Pcap=len(rows) - 1)
            assert mk2["status"][0] == orc.ST_PATHS_TRUNCATED
            assert (mk2["retrieve"][0] == mk["retrieve"][0, :len(rows) - 1]).all()
            assert (mk2["dense"] == mk["dense"]).all()


def test_padding_and_ragged_batches_do_not_leak():
    rng = np.random.default_rng(4)
    Nmax = 24
    parent = np.zeros((3, Nmax), dtype=np.int32)
    n = np.array([24, 9, 1], dtype=np.int32)
    for b in range(3):
        parent[b, :n[b]] = random_parent_tree(int(n[b]), min(3, int(n[b]) - 1), rng) if n[b] > 1 else [-1]
    mk = orc.build_mask(parent, n, Dcap=3, Pcap=Nmax)
    garbage = parent.copy()
    for b in range(3):
        garbage[b, n[b]:] = rng.integers(-5, 99, size=Nmax - n[b])
    mk2 = orc.build_mask(garbage, n, Dcap=3, Pcap=Nmax)
    for k in mk:
        assert (mk[k] == mk2[k]).all(), k
    for b in range(3):
        assert (mk["dense"][b, 0, n[b]:, :] == 0).all() and (mk["dense"][b, 0, :, n[b]:] == 0).all()
        assert (mk["depth"][b, n[b]:] == 0).all()


@pytest.mark.parametrize("bad", ["root", "range_hi", "range_neg", "order", "self", "depth", "n0"])
def test_malformed_trees_are_flagged_and_zeroed(bad):
    parent = np.array([[-1, 0, 1, 2, 3, 1]], dtype=np.int32)
    n, Dcap = np.array([6]), 4
    if bad == "root":
        parent[0, 0] = 0
    elif bad == "range_hi":
        parent[0, 3] = 6
    elif bad == "range_neg":
        parent[0, 3] = -1
    elif bad == "order":
        parent[0, 2] = 4
    elif bad == "self":
        parent[0, 2] = 2
    elif bad == "depth":
        Dcap = 3
    elif bad == "n0":
        n = np.array([0])
    mk = orc.build_mask(parent, n, Dcap=Dcap, Pcap=4)
    assert mk["status"][0] == orc.ST_BAD_TREE
    assert not mk["dense"].any() and not mk["anc_bits"].any() and not mk["depth"].any()
    assert (mk["retrieve"] == -1).all() and mk["n_paths"][0] == 0


# ------------------------------------------------------------- attention ----
def _attn_inputs(rng_seed, B, Hq, Hkv, d, Scap, Nmax, std=1.0):
    gen = torch.Generator().manual_seed(rng_seed)
    t = lambda *s: bf16_bits(randn_bf16(s, std, gen, "cpu"))
    return (t(B, Nmax, Hq, d), t(B, Hkv, Scap, d), t(B, Hkv, Scap, d),
            t(B, Nmax, Hkv, d), t(B, Nmax, Hkv, d))


def _softmax_attend(qv, ks, vs, scale):
    """Ordinary attention of one query over a key/value list, pure Python sums."""
    x = [scale * sum(float(a) * float(b) for a, b in zip(qv, k)) for k in ks]
    m = max(x)
    w = [math.exp(v - m) for v in x]
    l = sum(w)
    out = [sum(w[t] * float(vs[t][c]) for t in range(len(ks))) / l for c in range(len(vs[0]))]
    return out, m + math.log(l)


def test_attention_per_path_brute_force():
    """Row i equals causal attention of the last token of prefix (+) path(i)."""
    rng = np.random.default_rng(5)
    B, Hq, Hkv, d, Scap, N = 2, 4, 2, 8, 12, 9
    q, kc, vc, kt, vt = _attn_inputs(11, B, Hq, Hkv, d, Scap, N)
    parent = np.stack([random_parent_tree(N, 3, rng), random_parent_tree(N, 4, rng)])
    n = np.array([N, N - 2], dtype=np.int32)
    parent[1, N - 2:] = 0
    parent[1, :N - 2] = random_parent_tree(N - 2, 3, rng)
    S = np.array([5, 0], dtype=np.int32)
    mk = orc.build_mask(parent, n, Dcap=4, Pcap=N)
    scale = 0.37
    out, lse = orc.tree_attention(q, kc, vc, kt, vt, S, n, mk["dense"][:, 0], scale)
    f = orc.decode_bf16
    for b in range(B):
        for i in range(N):
            for h in range(Hq):
                if i >= n[b]:
                    assert (out[b, i, h] == 0).all() and lse[b, h, i] == -np.inf
                    continue
                hk = h // (Hq // Hkv)
                path = sorted(_anc_set_by_walk(parent[b], i))
                ks = [f(kc[b, hk, s]) for s in range(S[b])] + [f(kt[b, j, hk]) for j in path]
                vs = [f(vc[b, hk, s]) for s in range(S[b])] + [f(vt[b, j, hk]) for j in path]
                o, l = _softmax_attend(f(q[b, i, h]), ks, vs, scale)
                assert np.allclose(out[b, i, h], o, rtol=0, atol=1e-12)
                assert abs(lse[b, h, i] - l) < 1e-12


def test_attention_matches_library_sdpa_general_and_special_trees():
    """torch SDPA in fp64 with a boolean mask built by parent walks (general
    tree), a chain tree (bottom-right aligned causal attention) and a 1-node
    tree (single-token decode)."""
    rng = np.random.default_rng(6)
    B, Hq, Hkv, d, Scap = 1, 4, 2, 16, 40
    for N, parent in [(13, random_parent_tree(13, 4, rng)), (10, chain_tree(10)), (1, chain_tree(1))]:
        q, kc, vc, kt, vt = _attn_inputs(100 + N, B, Hq, Hkv, d, Scap, N)
        S = np.array([33], dtype=np.int32)
        n = np.array([N], dtype=np.int32)
        mk = orc.build_mask(parent[None], n, Dcap=N, Pcap=N)
        out, _ = orc.tree_attention(q, kc, vc, kt, vt, S, n, mk["dense"][:, 0], 0.25)
        allow = torch.zeros(N, S[0] + N, dtype=torch.bool)
        allow[:, :S[0]] = True
        for i in range(N):
            for j in _anc_set_by_walk(parent, i):
                allow[i, S[0] + j] = True
        if N == 10:   # chain: the textbook causal triangle, bottom-right aligned
            assert torch.equal(allow, torch.ones(N, S[0] + N).tril(diagonal=int(S[0])).bool())
        tq = torch.from_numpy(orc.decode_bf16(q))[0].permute(1, 0, 2)                     # [Hq,N,d]
        G = Hq // Hkv
        tk = torch.cat([torch.from_numpy(orc.decode_bf16(kc))[0, :, :S[0]],
                        torch.from_numpy(orc.decode_bf16(kt))[0].permute(1, 0, 2)], 1).repeat_interleave(G, 0)
        tv = torch.cat([torch.from_numpy(orc.decode_bf16(vc))[0, :, :S[0]],
                        torch.from_numpy(orc.decode_bf16(vt))[0].permute(1, 0, 2)], 1).repeat_interleave(G, 0)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=allow, scale=0.25)
        assert np.allclose(out[0], ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_attention_closed_forms():
    """K = 0 => lse = ln(S + depth + 1) and out = mean of the visible V rows;
    all V rows equal c => out = c."""
    rng = np.random.default_rng(7)
    B, Hq, Hkv, d, Scap, N = 1, 2, 1, 4, 20, 11
    parent = random_parent_tree(N, 4, rng)
    n = np.array([N])
    mk = orc.build_mask(parent[None], n, Dcap=4, Pcap=N)
    q, kc, vc, kt, vt = _attn_inputs(21, B, Hq, Hkv, d, Scap, N)
    for S0 in (0, 1, 16):
        S = np.array([S0], dtype=np.int32)
        out, lse = orc.tree_attention(q, np.zeros_like(kc), vc, np.zeros_like(kt), vt, S, n,
                                      mk["dense"][:, 0], 1.0)
        for i in range(N):
            anc = sorted(_anc_set_by_walk(parent, i))
            assert abs(lse[0, 0, i] - math.log(S0 + mk["depth"][0, i] + 1)) < 1e-12
            mean = (orc.decode_bf16(vc[0, 0, :S0]).sum(0) + orc.decode_bf16(vt[0, anc, 0]).sum(0)) / (S0 + len(anc))
            assert np.allclose(out[0, i, 0], mean, atol=1e-12)
    c = _bf16(np.arange(d) - 1.5)
    vcc = np.broadcast_to(c, vc.shape).copy()
    vtc = np.broadcast_to(c, vt.shape).copy()
    out, _ = orc.tree_attention(q, kc, vcc, kt, vtc, np.array([7]), n, mk["dense"][:, 0], 0.5)
    assert np.allclose(out[0], np.arange(d) - 1.5, atol=1e-12)


def test_attention_non_ancestor_perturbation_and_stale_cache_rows():
    rng = np.random.default_rng(8)
    B, Hq, Hkv, d, Scap, N = 1, 2, 2, 8, 16, 12
    parent = random_parent_tree(N, 3, rng)
    n = np.array([N])
    mk = orc.build_mask(parent[None], n, Dcap=3, Pcap=N)
    q, kc, vc, kt, vt = _attn_inputs(31, B, Hq, Hkv, d, Scap, N)
    S = np.array([6], dtype=np.int32)
    out, lse = orc.tree_attention(q, kc, vc, kt, vt, S, n, mk["dense"][:, 0], 0.3)
    victim = N - 1
    kt2, vt2 = kt.copy(), vt.copy()
    kt2[0, victim] = _bf16(np.full((Hkv, d), 50.0))
    vt2[0, victim] = _bf16(np.full((Hkv, d), -77.0))
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[0, :, 6:] = 0x7FC0      # NaN in the rows past the prefix: ignored by definition
    vc2[0, :, 6:] = 0x7FC0
    out2, lse2 = orc.tree_attention(q, kc2, vc2, kt2, vt2, S, n, mk["dense"][:, 0], 0.3)
    anc_of = lambda i: _anc_set_by_walk(parent, i)
    for i in range(N):
        if victim not in anc_of(i):
            assert (out[0, i] == out2[0, i]).all() and (lse[0, :, i] == lse2[0, :, i]).all()
        else:
            assert not np.allclose(out[0, i], out2[0, i])
    assert np.isfinite(out2).all()


# ---------------------------------------------------- gather / argmax / accept
def test_safe_gather_brute_force_and_sentinel_independence():
    rng = np.random.default_rng(9)
    B, P, Dp1, N = 3, 6, 5, 10
    n = np.array([10, 7, 4])
    retrieve = rng.integers(-1, 4, size=(B, P, Dp1)).astype(np.int32)
    tokens = rng.integers(0, 1000, size=(B, N)).astype(np.int32)
    safe, cand, ok, st = orc.safe_gather(retrieve, tokens, n)
    assert (st == 0).all()
    assert safe.min() >= 0 and (safe < n[:, None, None]).all()
    assert (safe == np.where(retrieve < 0, 0, retrieve)).all()
    assert (cand == np.take_along_axis(tokens, safe.reshape(B, -1), 1).reshape(B, P, Dp1)).all()
    assert (ok == (retrieve >= 0)).all()
    # any other negative sentinel gives the same gather, plus the BAD_INDEX flag
    r2 = np.where(retrieve < 0, -9, retrieve)
    safe2, cand2, ok2, st2 = orc.safe_gather(r2, tokens, n)
    assert (safe2 == safe).all() and (cand2 == cand).all() and (ok2 == ok).all()
    assert (st2 == orc.ST_BAD_INDEX).all()
    # indices at or past n_nodes are remapped and flagged
    r3 = retrieve.copy()
    r3[2, 0, 0] = 4
    safe3, _, ok3, st3 = orc.safe_gather(r3, tokens, n)
    assert safe3[2, 0, 0] == 0 and not ok3[2, 0, 0] and st3.tolist() == [0, 0, orc.ST_BAD_INDEX]


def test_argmax_matches_numpy_first_occurrence_with_planted_ties():
    rng = np.random.default_rng(10)
    B, N, V = 2, 5, 4096
    x = rng.standard_normal((B, N, V)).astype(np.float32)
    bits = _bf16(x)
    top = np.uint16(0x4120)   # 10.0
    bits[0, 1, [77, 900, 4000]] = top
    bits[1, 2, [4095, 5]] = top
    bits[1, 3, :] = 0x8000                # all -0.0 ...
    bits[1, 3, 9] = 0x0000                # ... and one +0.0: they tie, lowest index wins
    n = np.array([5, 4])
    am = orc.argmax_rows(bits, n)
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    want = np.argmax(wide, axis=-1)       # numpy documents first occurrence
    assert (am[0] == want[0]).all() and (am[1, :4] == want[1, :4]).all()
    assert am[0, 1] == 77 and am[1, 2] == 5 and am[1, 3] == 0 and am[1, 4] == -1


def _walk_accept(parent, n, tokens, am):
    """Tree-walk formulation: from the root follow the child whose token equals
    the teacher's argmax at the current node (children have distinct tokens)."""
    cur, nodes = 0, [0]
    while True:
        nxt = [c for c in range(1, n) if parent[c] == cur and tokens[c] == am[cur]]
        if not nxt:
            return nodes
        cur = nxt[0]
        nodes.append(cur)


def test_accept_equals_tree_walk_and_planted_depths():
    rng = np.random.default_rng(11)
    for trial in range(30):
        N, D = 40, 6
        parent = topk_expansion_tree(N, D, 5, rng)
        rows = leaf_paths(parent)
        V = 50 if trial % 2 else 100000
        tokens = np.zeros(N, dtype=np.int32)
        for p in range(N):      # distinct tokens among siblings
            kids = [c for c in range(1, N) if parent[c] == p]
            tokens[kids] = rng.choice(V, size=len(kids), replace=False)
        am = rng.integers(0, V, size=N).astype(np.int32)
        deepest = max(rows, key=len)
        a = int(rng.integers(0, len(deepest)))
        for j in range(1, a + 1):
            am[deepest[j - 1]] = tokens[deepest[j]]
        if a < len(deepest) - 1:     # stop exactly there
            kids = [c for c in range(1, N) if parent[c] == deepest[a]]
            am[deepest[a]] = V + 1
        retrieve = np.full((1, len(rows), D + 1), -1, dtype=np.int32)
        for p, r in enumerate(rows):
            retrieve[0, p, :len(r)] = r
        acc = orc.greedy_accept(retrieve, tokens[None], np.array([N]), am[None])
        walk = _walk_accept(parent, N, tokens, am)
        assert walk == deepest[:a + 1]
        assert acc["accept_len"][0] == a == len(walk) - 1
        assert acc["accepted_nodes"][0, :a + 1].tolist() == walk
        assert (acc["accepted_nodes"][0, a + 1:] == 0).all()
        assert acc["next_token"][0] == am[walk[-1]]
        first = min(p for p, r in enumerate(rows) if r[:a + 1] == walk)
        assert acc["best_path"][0] == first          # lowest row among ties


def test_accept_dummy_index_cannot_over_accept():
    """The remapped slot points at node 0, whose token is real: without the
    validity guard a short row would accept past its leaf."""
    parent = np.array([[-1, 0, 1]], dtype=np.int32)
    tokens = np.array([[42, 5, 6]], dtype=np.int32)
    am = np.array([[5, 6, 42]], dtype=np.int32)      # am[leaf] == tokens[0]
    retrieve = np.array([[[0, 1, 2, -1, -1]]], dtype=np.int32)
    acc = orc.greedy_accept(retrieve, tokens, np.array([3]), am)
    assert acc["accept_len"][0] == 2 and acc["accepted_nodes"][0].tolist() == [0, 1, 2, 0, 0]
    assert acc["next_token"][0] == 42
    # no candidate rows at all: accept nothing, commit the root, bonus = am[root]
    acc = orc.greedy_accept(np.full((1, 2, 5), -1, dtype=np.int32), tokens, np.array([3]), am)
    assert acc["accept_len"][0] == 0 and acc["accepted_nodes"][0].tolist() == [0] * 5
    assert acc["next_token"][0] == 5


def test_random_tokens_with_large_vocab_accept_nothing():
    rng = np.random.default_rng(12)
    N, D = 30, 5
    parent = topk_expansion_tree(N, D, 4, rng)
    rows = leaf_paths(parent)
    retrieve = np.full((1, len(rows), D + 1), -1, dtype=np.int32)
    for p, r in enumerate(rows):
        retrieve[0, p, :len(r)] = r
    tokens = rng.integers(0, 2 ** 30, size=(1, N)).astype(np.int32)
    am = rng.integers(0, 2 ** 30, size=(1, N)).astype(np.int32)
    acc = orc.greedy_accept(retrieve, tokens, np.array([N]), am)
    assert acc["accept_len"][0] == 0 and acc["best_path"][0] == 0


# ----------------------------------------------------------------- commit ----
def test_commit_bytes_and_untouched_regions():
    rng = np.random.default_rng(13)
    L, B, Hkv, Scap, d, N, Dp1 = 3, 3, 2, 20, 4, 7, 4
    kc = rng.integers(0, 2 ** 16, size=(L, B, Hkv, Scap, d)).astype(np.uint16)
    vc = rng.integers(0, 2 ** 16, size=(L, B, Hkv, Scap, d)).astype(np.uint16)
    kt = rng.integers(0, 2 ** 16, size=(L, B, N, Hkv, d)).astype(np.uint16)
    vt = rng.integers(0, 2 ** 16, size=(L, B, N, Hkv, d)).astype(np.uint16)
    nodes = np.array([[0, 2, 5, 0], [0, 0, 0, 0], [0, 1, 3, 6]], dtype=np.int32)
    A = np.array([2, 0, 3], dtype=np.int32)
    S = np.array([10, 0, 17], dtype=np.int32)      # third one overflows: 17+4 > 20
    kc2, vc2, S2, st = orc.kv_commit(kc, vc, kt, vt, nodes, A, S)
    assert st.tolist() == [0, 0, orc.ST_CAPACITY]
    assert S2.tolist() == [13, 1, 17]
    want_k, want_v = kc.copy(), vc.copy()
    want_k[:, 0, :, 10:13] = kt[:, 0, [0, 2, 5]].transpose(0, 2, 1, 3)
    want_v[:, 0, :, 10:13] = vt[:, 0, [0, 2, 5]].transpose(0, 2, 1, 3)
    want_k[:, 1, :, 0:1] = kt[:, 1, [0]].transpose(0, 2, 1, 3)
    want_v[:, 1, :, 0:1] = vt[:, 1, [0]].transpose(0, 2, 1, 3)
    assert (kc2 == want_k).all() and (vc2 == want_v).all()
    # fatal incoming status and bad node ids skip the sequence
    _, _, S3, st3 = orc.kv_commit(kc, vc, kt, vt, nodes, A, S, status_in=np.array([orc.ST_BAD_TREE, 0, 0]))
    assert S3.tolist() == [10, 1, 17] and st3[0] == orc.ST_BAD_TREE
    bad = nodes.copy()
    bad[0, 1] = 7
    kc4, _, S4, st4 = orc.kv_commit(kc, vc, kt, vt, bad, A, S)
    assert st4[0] == orc.ST_BAD_INDEX and S4[0] == 10 and (kc4[:, 0] == kc[:, 0]).all()


def test_commit_equivalence_with_sequential_decoding():
    """After the commit, a 1-node verify equals plain causal decode over
    prefix (+) accepted path; a chain tree makes the path commit the
    length-based commit."""
    rng = np.random.default_rng(14)
    B, Hq, Hkv, d, Scap, N = 1, 2, 1, 8, 24, 9
    parent = random_parent_tree(N, 4, rng)
    q, kc, vc, kt, vt = _attn_inputs(41, B, Hq, Hkv, d, Scap, N)
    rows = leaf_paths(parent)
    path = max(rows, key=len)
    A = len(path) - 1
    nodes = np.zeros((1, 5), dtype=np.int32)
    nodes[0, :A + 1] = path
    S = np.array([7], dtype=np.int32)
    kc2, vc2, S2, st = orc.kv_commit(kc[None], vc[None], kt[None], vt[None], nodes, np.array([A]), S)
    assert st[0] == 0 and S2[0] == 7 + A + 1
    q1, _, _, kt1, vt1 = _attn_inputs(43, B, Hq, Hkv, d, Scap, 1)
    mk1 = orc.build_mask(np.array([[-1]]), np.array([1]), Dcap=0, Pcap=1)
    out, _ = orc.tree_attention(q1, kc2[0], vc2[0], kt1, vt1, S2, np.array([1]), mk1["dense"][:, 0], 0.4)
    f = orc.decode_bf16
    ks = [f(kc[0, 0, s]) for s in range(7)] + [f(kt[0, j, 0]) for j in path] + [f(kt1[0, 0, 0])]
    vs = [f(vc[0, 0, s]) for s in range(7)] + [f(vt[0, j, 0]) for j in path] + [f(vt1[0, 0, 0])]
    for h in range(Hq):
        o, _ = _softmax_attend(f(q1[0, 0, h]), ks, vs, 0.4)
        assert np.allclose(out[0, 0, h], o, atol=1e-12)
    # chain tree: accepted_nodes = 0..A is "keep the first A new steps"
    nodes_c = np.arange(5, dtype=np.int32)[None]
    kc3, _, _, _ = orc.kv_commit(kc[None], vc[None], kt[None], vt[None], nodes_c, np.array([3]), S)
    assert (kc3[0, 0, :, 7:11] == kt[0, 0:4].transpose(1, 0, 2)).all()


def test_inplace_commit_worked_example_with_overlapping_rows():
    """Full reorder inside the cache: the expected rows are typed out by hand.  Rows carry their own
    index as content (row r holds the value 100 + r), prefix 3, tree of 6 nodes at rows 3..8, accepted
    path {0, 2, 3}: row 5 (node 2) is the source of slot 1 AND the destination of slot 2, so a copy
    that writes slot 2 before it reads slot 1's source would put 106 into row 4."""
    L, B, Hkv, Scap, d, N = 1, 1, 1, 10, 2, 6
    kc = np.zeros((L, B, Hkv, Scap, d), dtype=np.uint16)
    kc[0, 0, 0, :, 0] = 100 + np.arange(Scap)
    kc[0, 0, 0, :, 1] = 200 + np.arange(Scap)
    vc = kc + 1000
    nodes = np.array([[0, 2, 3, 0]], dtype=np.int32)
    kc2, vc2, S2, st = orc.kv_commit_inplace(kc, vc, nodes, np.array([2]), np.array([3]), N)
    assert st.tolist() == [0] and S2.tolist() == [6]
    #            prefix rows 0..2   | slot0 = node0 (row 3) | slot1 = node2 (row 5) | slot2 = node3 (row 6) | stale rows
    assert kc2[0, 0, 0, :, 0].tolist() == [100, 101, 102, 103, 105, 106, 106, 107, 108, 109]
    assert kc2[0, 0, 0, :, 1].tolist() == [200, 201, 202, 203, 205, 206, 206, 207, 208, 209]
    assert (vc2 == kc2 + 1000).all()
    # a descending path order (not produced by a tree, but allowed by the definition) is still a gather
    # from the old state: slot 1 <- old row 3+3, slot 2 <- old row 3+1
    nodes = np.array([[0, 3, 1, 0]], dtype=np.int32)
    kc3, _, _, _ = orc.kv_commit_inplace(kc, vc, nodes, np.array([2]), np.array([3]), N)
    assert kc3[0, 0, 0, :, 0].tolist() == [100, 101, 102, 103, 106, 104, 106, 107, 108, 109]


def test_inplace_commit_equals_separate_buffer_commit_and_flags():
    """With the tree's rows placed behind the prefix, the in-cache reorder and the separate-buffer
    commit give the same committed rows [0, S+A+1); a chain path is the identity (length-based commit);
    capacity and index errors skip the sequence."""
    rng = np.random.default_rng(15)
    L, B, Hkv, Scap, d, N, Dp1 = 2, 3, 2, 24, 4, 7, 4
    kt = rng.integers(0, 2 ** 16, size=(L, B, N, Hkv, d)).astype(np.uint16)
    vt = rng.integers(0, 2 ** 16, size=(L, B, N, Hkv, d)).astype(np.uint16)
    kc = rng.integers(0, 2 ** 16, size=(L, B, Hkv, Scap, d)).astype(np.uint16)
    vc = rng.integers(0, 2 ** 16, size=(L, B, Hkv, Scap, d)).astype(np.uint16)
    S = np.array([10, 0, 17], dtype=np.int32)
    kin, vin = kc.copy(), vc.copy()
    for b in range(B):                                   # the forward pass extended the cache in place
        kin[:, b, :, S[b]:S[b] + N] = kt[:, b].transpose(0, 2, 1, 3)
        vin[:, b, :, S[b]:S[b] + N] = vt[:, b].transpose(0, 2, 1, 3)
    nodes = np.array([[0, 2, 5, 0], [0, 1, 2, 3], [0, 1, 3, 6]], dtype=np.int32)
    A = np.array([2, 3, 3], dtype=np.int32)
    k1, v1, S1, st1 = orc.kv_commit(kc, vc, kt, vt, nodes, A, S)
    k2, v2, S2, st2 = orc.kv_commit_inplace(kin, vin, nodes, A, S, N)
    assert st1.tolist() == st2.tolist() == [0, 0, 0] and S1.tolist() == S2.tolist() == [13, 4, 21]
    for b in range(B):
        assert (k1[:, b, :, :S1[b]] == k2[:, b, :, :S2[b]]).all() and (v1[:, b, :, :S1[b]] == v2[:, b, :, :S2[b]]).all()
        assert (k2[:, b, :, S2[b]:] == kin[:, b, :, S2[b]:]).all()        # rows behind the segment untouched
    assert (k2[:, 1] == kin[:, 1]).all()                                   # chain path: nothing moves
    # a source row past the capacity, a bad node id, a fatal incoming status
    _, _, S3, st3 = orc.kv_commit_inplace(kin, vin, nodes, A, np.array([10, 0, 18], dtype=np.int32), N)
    assert st3.tolist() == [0, 0, orc.ST_CAPACITY] and S3[2] == 18
    bad = nodes.copy()
    bad[0, 1] = N
    k4, _, S4, st4 = orc.kv_commit_inplace(kin, vin, bad, A, S, N, status_in=np.array([0, orc.ST_BAD_TREE, 0]))
    assert st4.tolist() == [orc.ST_BAD_INDEX, orc.ST_BAD_TREE, 0] and S4.tolist() == [10, 0, 21]
    assert (k4[:, :2] == kin[:, :2]).all()


def test_paged_cache_is_the_contiguous_cache_behind_a_block_table():
    """Layout pins: a hand-typed two-page example of the row mapping, and the paged commit equal to the
    contiguous commit seen through the block table (sequences own disjoint pages; a segment that crosses a
    page boundary; untouched pages stay untouched; bad page id, capacity)."""
    pages = np.zeros((3, 1, orc.PAGE_ROWS, 1), dtype=np.uint16)
    for pg in range(3):
        pages[pg, 0, :, 0] = 1000 * pg + np.arange(orc.PAGE_ROWS)
    bt = np.array([[2, 0]], dtype=np.int32)
    flat = orc.paged_to_contiguous(pages, bt)
    assert flat.shape == (1, 1, 256, 1)
    assert flat[0, 0, [0, 5, 127, 128, 130, 255], 0].tolist() == [2000, 2005, 2127, 0, 2, 127]

    rng = np.random.default_rng(16)
    L, B, Hkv, d, N, Dp1, n_pages, nb = 2, 3, 2, 4, 9, 4, 10, 3
    u16 = lambda *s_: rng.integers(0, 2 ** 16, size=s_).astype(np.uint16)
    kp, vp = u16(L, n_pages, Hkv, orc.PAGE_ROWS, d), u16(L, n_pages, Hkv, orc.PAGE_ROWS, d)
    kt, vt = u16(L, B, N, Hkv, d), u16(L, B, N, Hkv, d)
    bt = np.array([[7, 2, 9], [0, 5, 1], [3, 8, 4]], dtype=np.int32)      # page 6 belongs to nobody
    nodes = np.array([[0, 2, 5, 8], [0, 1, 0, 0], [0, 3, 4, 0]], dtype=np.int32)
    A = np.array([3, 1, 2], dtype=np.int32)
    S = np.array([126, 0, 381], dtype=np.int32)          # b=0 crosses pages 7 -> 2; b=2 ends exactly at the capacity 384
    kp2, vp2, S2, st = orc.kv_commit_paged(kp, vp, bt, kt, vt, nodes, A, S)
    assert st.tolist() == [0, 0, 0] and S2.tolist() == [130, 2, 384]
    cont = lambda pgs: np.stack([orc.paged_to_contiguous(pgs[l], bt) for l in range(L)])
    rk, rv, rS, rst = orc.kv_commit(cont(kp), cont(vp), kt, vt, nodes, A, S)
    assert (cont(kp2) == rk).all() and (cont(vp2) == rv).all() and rS.tolist() == S2.tolist()
    assert (kp2[:, 6] == kp[:, 6]).all() and (vp2[:, 6] == vp[:, 6]).all()
    assert (kp2[:, 7, :, 126] == kt[:, 0, 0]).all() and (kp2[:, 2, :, 1] == kt[:, 0, 8]).all()
    bad_bt = bt.copy()
    bad_bt[0, 1] = n_pages                                # the page the segment of b=0 runs into
    kp3, _, S3, st3 = orc.kv_commit_paged(kp, vp, bad_bt, kt, vt, nodes, A, np.array([126, 0, 382], dtype=np.int32))
    assert st3.tolist() == [orc.ST_BAD_INDEX, 0, orc.ST_CAPACITY] and S3.tolist() == [126, 2, 382]
    assert (kp3[:, 7] == kp[:, 7]).all()


# ---------------------------------------------------- sampling-mode acceptance ----
def _stoch_case():
    """V = 4, logits [2,1,0,0] in every row and T = 1/ln 2, so that p = [1/2, 1/4, 1/8, 1/8] exactly.
    Tree: root 0 -> node 1 (token 1), node 2 (token 0); node 2 -> node 3 (token 3)."""
    logits = _bf16(np.tile(np.array([2.0, 1.0, 0.0, 0.0], dtype=np.float32), (1, 4, 1)))
    tokens = np.array([[9, 1, 0, 3]], dtype=np.int32)
    parent = np.array([[-1, 0, 0, 2]], dtype=np.int32)
    return logits, tokens, parent, np.array([4]), 1.0 / np.log(2.0)


def test_stochastic_accept_hand_worked_example():
    logits, tokens, parent, n, T = _stoch_case()
    run = lambda un, ub: orc.stochastic_accept(logits, tokens, parent, n, np.array([un]), np.array([ub]), T, 4)
    # root: node 1 (p = 1/4) fails at u = 0.3; node 2 has p = (1/2)/(3/4) = 2/3 and passes at 0.5; node 3 (p = 1/8)
    # passes at 0.1; leaf: token from [1/2, 3/4, 7/8, 1] at 0.6 -> 1
    r = run([0.0, 0.3, 0.5, 0.1], 0.6)
    assert r["accept_len"].tolist() == [2] and r["accepted_nodes"].tolist() == [[0, 2, 3, 0]] and r["next_token"].tolist() == [1]
    # node 2 fails at 0.7 > 2/3: tokens 1 and 0 are out, the rest is [0, 0, 1/2, 1/2]
    r = run([0.0, 0.3, 0.7, 0.1], 0.4)
    assert r["accept_len"].tolist() == [0] and r["accepted_nodes"].tolist() == [[0, 0, 0, 0]] and r["next_token"].tolist() == [2]
    assert run([0.0, 0.3, 0.7, 0.1], 0.5)["next_token"].tolist() == [3]
    assert run([0.0, 0.3, 0.7, 0.1], 0.0)["next_token"].tolist() == [2]       # never a rejected token, even at u = 0
    # node 1 passes at once; it has no children: token drawn from the unmodified p
    r = run([0.0, 0.2, 0.9, 0.9], 0.49)
    assert r["accept_len"].tolist() == [1] and r["accepted_nodes"].tolist() == [[0, 1, 0, 0]] and r["next_token"].tolist() == [0]
    # capacity of the accepted list: Dp1 = 2 keeps one accepted node and then samples at it
    r = orc.stochastic_accept(logits, tokens, parent, n, np.array([[0.0, 0.3, 0.5, 0.0]]), np.array([0.8]), T, 2)
    assert r["accept_len"].tolist() == [1] and r["accepted_nodes"].tolist() == [[0, 2]] and r["next_token"].tolist() == [2]
    # a proposed token outside the vocabulary is never accepted and is reported
    bad = tokens.copy()
    bad[0, 1] = 4
    r = orc.stochastic_accept(logits, bad, parent, n, np.array([[0.0, 0.0, 0.4, 0.9]]), np.array([0.1]), T, 4)
    assert r["status"].tolist() == [orc.ST_BAD_INDEX] and r["accepted_nodes"].tolist() == [[0, 2, 0, 0]]
    # The flag is a property of the inputs, not of the walk: every valid non-root slot is checked, also one the walk
    # never tries (node 3 hangs under node 2, which fails here) - the same rule as for the candidate rows of the
    # greedy gather, where an out-of-range index in any slot is reported whether or not acceptance reaches it.
    untried = tokens.copy()
    untried[0, 3] = 99
    r = orc.stochastic_accept(logits, untried, parent, n, np.array([[0.0, 0.3, 0.7, 0.1]]), np.array([0.4]), T, 4)
    assert r["status"].tolist() == [orc.ST_BAD_INDEX]
    assert r["accept_len"].tolist() == [0] and r["next_token"].tolist() == [2]       # the walk itself is unchanged
    # a padded slot (here slot 3, with three active nodes) is not a proposal and raises nothing
    r = orc.stochastic_accept(logits, untried, parent, np.array([3]), np.array([[0.0, 0.3, 0.7, 0.1]]), np.array([0.4]), T, 4)
    assert r["status"].tolist() == [0]


def test_stochastic_accept_becomes_greedy_at_low_temperature():
    rng = np.random.default_rng(31)
    B, N, V, D = 3, 14, 50, 4
    parent = np.stack([random_parent_tree(N, D, rng) for _ in range(B)])
    n = np.array([N, N, 9])
    vals = rng.standard_normal((B, N, V)).astype(np.float32)
    for b in range(B):
        for i in range(N):
            vals[b, i, rng.integers(V)] = 6.0                  # a unique maximum per row
    bits = _bf16(vals)
    am = orc.argmax_rows(bits, n)
    tokens = rng.integers(0, V, size=(B, N)).astype(np.int32)
    for b in range(B):                                          # let some children carry the teacher's token
        for k in range(1, int(n[b])):
            if rng.random() < 0.6:
                tokens[b, k] = am[b, parent[b, k]]
    u = rng.random((B, N))
    r = orc.stochastic_accept(bits, tokens, parent, n, u, rng.random(B), 1e-3, D + 1)
    for b in range(B):                                          # the greedy walk: follow the child that carries the argmax
        c, path = 0, [0]
        while len(path) < D + 1:
            nxt = [k for k in range(c + 1, int(n[b])) if parent[b, k] == c and tokens[b, k] == am[b, c]]
            if not nxt:
                break
            c = nxt[0]
            path.append(c)
        assert r["accept_len"][b] == len(path) - 1 and r["accepted_nodes"][b, :len(path)].tolist() == path
        assert r["next_token"][b] == am[b, c]


def test_stochastic_accept_first_token_follows_the_teacher_distribution():
    """The property the rule exists for: whatever the tree proposes (here with a duplicated sibling token and
    a zero-probability-ish one), the first token that leaves the step is distributed as softmax(logits/T)
    at the root.  30000 draws, every probability within 4.5 standard errors."""
    rng = np.random.default_rng(32)
    V, T = 6, 0.9
    row = np.array([1.5, 0.25, 1.0, -2.0, 0.5, 0.0], dtype=np.float32)
    bits = _bf16(np.tile(row, (1, 6, 1)))
    tokens = np.array([[0, 2, 4, 2, 3, 1]], dtype=np.int32)       # children of the root: 2, 4, 2 (again), 3; node 5 under node 1
    parent = np.array([[-1, 0, 0, 0, 0, 1]], dtype=np.int32)
    n = np.array([6])
    p = np.exp(orc.decode_bf16(bits[0, 0]).astype(np.float64) / T)
    p /= p.sum()
    draws = 30000
    counts = np.zeros(V)
    accepted = 0
    for _ in range(draws):
        r = orc.stochastic_accept(bits, tokens, parent, n, rng.random((1, 6)), rng.random(1), T, 3)
        if r["accept_len"][0] >= 1:
            counts[tokens[0, r["accepted_nodes"][0, 1]]] += 1
            accepted += 1
        else:
            counts[r["next_token"][0]] += 1
    se = np.sqrt(p * (1 - p) / draws)
    assert (np.abs(counts / draws - p) < 4.5 * se).all(), (counts / draws, p)
    assert 0.3 * draws < accepted < 0.9 * draws                  # both branches of the rule were exercised


def test_node_scores_gather_and_link_to_greedy_acceptance():
    """score[k] = logits[parent(k), token(k)]: checked against numpy fancy indexing, and against the
    acceptance rule - a node is accepted by the greedy rule exactly when its score equals the row
    maximum at its parent and its token is the lowest maximiser."""
    rng = np.random.default_rng(21)
    B, N, V = 2, 12, 300
    parent = np.stack([random_parent_tree(N, 4, rng), random_parent_tree(N, 3, rng)])
    n = np.array([N, 9])
    bits = _bf16(rng.standard_normal((B, N, V)).astype(np.float32))
    tokens = rng.integers(0, V, size=(B, N)).astype(np.int32)
    am = orc.argmax_rows(bits, n)
    for b in range(B):                        # make some nodes match the teacher
        for k in (1, 3, 5):
            tokens[b, k] = am[b, max(parent[b, k], 0)]
    scores, st = orc.node_scores(bits, tokens, parent, n)
    assert (st == 0).all()
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    for b in range(B):
        sp = np.maximum(parent[b], 0)
        want = wide[b, sp, tokens[b]]
        want[0] = 0
        want[n[b]:] = 0
        assert np.array_equal(scores[b], want)
        for k in range(1, n[b]):
            is_top = scores[b, k] == wide[b, sp[k]].max()
            assert (tokens[b, k] == am[b, sp[k]]) == (is_top and tokens[b, k] == np.flatnonzero(wide[b, sp[k]] == wide[b, sp[k]].max())[0])
    bad = tokens.copy()
    bad[1, 2] = V
    bad[0, 4] = -3
    s2, st2 = orc.node_scores(bits, bad, parent, n)
    assert st2.tolist() == [orc.ST_BAD_INDEX] * 2 and np.isneginf(s2[1, 2]) and np.isneginf(s2[0, 4])


def test_merge_partials_equals_attention_over_the_union_of_key_ranges():
    """Pin for merge_partials: splitting the committed prefix in R ranges, attending to each range
    separately (tree keys with the last range only) and merging must give the attention over all
    keys - an identity of the softmax, so the two oracle results agree to rounding."""
    rng = np.random.default_rng(11)
    B, Hq, Hkv, d, N, Scap = 2, 4, 2, 8, 6, 40
    f = lambda *s: _bf16(rng.standard_normal(s).astype(np.float32))
    q, kc, vc = f(B, N, Hq, d), f(B, Hkv, Scap, d), f(B, Hkv, Scap, d)
    kt, vt = f(B, N, Hkv, d), f(B, N, Hkv, d)
    S = np.array([37, 5])
    n = np.array([6, 4])
    parent = np.array([[-1, 0, 0, 1, 1, 2], [-1, 0, 1, 2, 0, 0]])
    vis = orc.build_mask(parent, n, 5, 1, emit_paths=False)["dense"][:, 0]
    full, full_lse = orc.tree_attention(q, kc, vc, kt, vt, S, n, vis, 0.3)
    for R in (1, 2, 3, 5):
        o_parts, l_parts = [], []
        for r in range(R):
            lo, hi = (S * r) // R, (S * (r + 1)) // R          # key range of "rank" r per sequence
            kc_r, vc_r = np.zeros_like(kc), np.zeros_like(vc)
            for b in range(B):
                kc_r[b, :, :hi[b] - lo[b]] = kc[b, :, lo[b]:hi[b]]
                vc_r[b, :, :hi[b] - lo[b]] = vc[b, :, lo[b]:hi[b]]
            vis_r = vis if r == R - 1 else np.zeros_like(vis)   # tree keys belong to the last range
            o, l = orc.tree_attention(q, kc_r, vc_r, kt, vt, hi - lo, n, vis_r, 0.3)
            o_parts.append(o)
            l_parts.append(l)
        out, lse = orc.merge_partials(np.stack(o_parts), np.stack(l_parts))
        assert np.allclose(out, full, rtol=0, atol=1e-12)
        assert np.array_equal(np.isneginf(lse), np.isneginf(full_lse))
        fin = np.isfinite(full_lse)
        assert np.allclose(lse[fin], full_lse[fin], rtol=0, atol=1e-12)
    # with R = 5 the short sequence (S = 5 -> ranges of 1 key) and padded rows exercise small and empty ranges


def test_merge_partials_closed_forms():
    """R = 1 is the identity; equal lse gives the plain average; an empty range (lse = -inf) is ignored even
    if its O holds NaN; all ranges empty gives zeros and -inf."""
    o = np.zeros((3, 1, 2, 1, 4))
    o[0, 0, 0, 0] = [1, 2, 3, 4]
    o[1, 0, 0, 0] = [3, 2, 1, 0]
    o[2] = np.nan
    l = np.full((3, 1, 1, 2), -np.inf)
    l[0, 0, 0, 0] = l[1, 0, 0, 0] = 0.7
    out, lse = orc.merge_partials(o, l)
    assert np.allclose(out[0, 0, 0], [2, 2, 2, 2]) and np.isclose(lse[0, 0, 0], 0.7 + np.log(2.0))
    assert (out[0, 1, 0] == 0).all() and lse[0, 0, 1] == -np.inf
    one, one_l = orc.merge_partials(o[:1], l[:1])
    assert np.array_equal(one[0, 0, 0], o[0, 0, 0, 0]) and one_l[0, 0, 0] == 0.7
    l[1, 0, 0, 0] = 0.7 + np.log(3.0)                      # weights 1 : 3
    out, lse = orc.merge_partials(o, l)
    assert np.allclose(out[0, 0, 0], (np.array([1, 2, 3, 4]) + 3 * np.array([3, 2, 1, 0])) / 4)
