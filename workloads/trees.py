"""Draft-tree generators (inputs only).

Trees are parent arrays over nodes 0..N-1 with node 0 the root
(``parent[0] = -1``) and ``parent[i] < i`` for every other node, the
linearisation of Section 3.2 with the root kept as row 0.  The paper gives
no draft-tree construction algorithm, so these are stand-ins with its
budgets and depth bounds (Table 2).
"""
import numpy as np


def _depths(parent):
    dep = np.zeros(len(parent), dtype=np.int64)
    for i in range(1, len(parent)):
        dep[i] = dep[parent[i]] + 1
    return dep


def random_parent_tree(N, D, rng):
    """parent[i] uniform in [0, i), redrawn while the parent already sits at
    depth D; the whole tree is redrawn until its maximum depth is exactly D."""
    assert N >= D + 1
    while True:
        parent = np.full(N, -1, dtype=np.int32)
        dep = np.zeros(N, dtype=np.int64)
        for i in range(1, N):
            while True:
                p = int(rng.integers(0, i))
                if dep[p] < D:
                    break
            parent[i] = p
            dep[i] = dep[p] + 1
        if dep.max() == D:
            return parent


def topk_expansion_tree(N, D, topk, rng):
    """EAGLE-style top-k expansion stand-in.

    Level 1 holds ``topk`` children of the root scored by -Exp(1) draws; every
    later level expands the ``topk`` best nodes of the previous level with
    ``topk`` children each (child score = parent score - Exp(1) draw).  After
    D levels the N-1 best-scoring candidates are kept (scores fall along a
    path, so the kept set is ancestor-closed) and renumbered in
    (level, score) order, which gives parent < child.  Redrawn until the kept
    tree has maximum depth D.
    """
    if N - 1 > topk + (D - 1) * topk * topk or N < D + 1:
        raise ValueError("node budget does not fit the expansion pool")
    while True:
        # candidate pool: (score, level, parent_candidate_id)
        score = [0.0]
        level = [0]
        par = [-1]
        frontier = [0]
        for lv in range(1, D + 1):
            new = []
            for f in frontier:
                for _ in range(topk):
                    score.append(score[f] - float(rng.exponential(1.0)))
                    level.append(lv)
                    par.append(f)
                    new.append(len(score) - 1)
            new.sort(key=lambda c: -score[c])
            frontier = new[:topk]
        cand = sorted(range(1, len(score)), key=lambda c: -score[c])[: N - 1]
        if len(cand) < N - 1:
            continue
        keep = [0] + sorted(cand, key=lambda c: (level[c], -score[c]))
        new_id = {c: i for i, c in enumerate(keep)}
        if any(par[c] not in new_id for c in keep[1:]):
            continue
        parent = np.array([-1] + [new_id[par[c]] for c in keep[1:]], dtype=np.int32)
        if _depths(parent).max() == D:
            return parent


def spine_tree(N, D, rng):
    """A tree that reaches depth D for any budget N > D: nodes 1..D form a chain from the root, every later
    node picks a uniform parent among the nodes of depth < D (deep, narrow budgets of the paper's sweep)."""
    assert N >= D + 1
    parent = np.full(N, -1, dtype=np.int32)
    dep = np.zeros(N, dtype=np.int64)
    for i in range(1, N):
        if i <= D:
            p = i - 1
        else:
            while True:
                p = int(rng.integers(0, i))
                if dep[p] < D:
                    break
        parent[i] = p
        dep[i] = dep[p] + 1
    return parent


def covering_chains_tree(N, n_chains, D, rng):
    """Chains hanging from the root whose root-to-leaf rows cover every node: N - 1 nodes spread over
    `n_chains` chains of depth <= D, as long as possible, the shorter ones at seeded positions (for N = 60,
    ten chains, D = 6: nine chains of depth 6 and one of depth 5 - the only kind of 60-node tree whose ten
    candidate rows of seven columns name all of its nodes).  Node ids run chain by chain."""
    assert n_chains >= 1 and n_chains <= N - 1 <= n_chains * D
    base, extra = divmod(N - 1, n_chains)
    lengths = np.full(n_chains, base, dtype=np.int64)
    lengths[rng.permutation(n_chains)[:extra]] += 1
    parent = np.full(N, -1, dtype=np.int32)
    i = 1
    for ln in lengths:
        for k in range(int(ln)):
            parent[i] = 0 if k == 0 else i - 1
            i += 1
    return parent


def chain_tree(N):
    """0 <- 1 <- 2 ... : the linear speculative proposal of Section 2.2."""
    return np.arange(-1, N - 1, dtype=np.int32)


def star_tree(N):
    """Every non-root node is a child of the root."""
    p = np.zeros(N, dtype=np.int32)
    p[0] = -1
    return p


def leaf_paths(parent, n_nodes=None):
    """All root-to-leaf node lists, leaves in increasing node id."""
    n = len(parent) if n_nodes is None else int(n_nodes)
    has_child = np.zeros(n, dtype=bool)
    for i in range(1, n):
        has_child[parent[i]] = True
    rows = []
    for leaf in range(n):
        if has_child[leaf]:
            continue
        chain = [leaf]
        while parent[chain[-1]] >= 0:
            chain.append(int(parent[chain[-1]]))
        rows.append(chain[::-1])
    return rows


def capped_paths(parent, P, first_leaf=None):
    """At most P candidate rows: ``first_leaf`` (if given) first, then the
    deepest remaining leaves, ties by lowest node id; the kept rows are
    sorted by leaf id."""
    rows = leaf_paths(parent)
    chosen = []
    if first_leaf is not None:
        chosen = [r for r in rows if r[-1] == first_leaf]
    rest = [r for r in rows if not chosen or r[-1] != chosen[0][-1]]
    rest.sort(key=lambda r: (-len(r), r[-1]))
    chosen = (chosen + rest)[:P]
    chosen.sort(key=lambda r: r[-1])
    return chosen


def rows_to_retrieve(rows, P, Dp1):
    """Left-aligned root-to-leaf rows, -1 after the leaf, all -1 past the last row."""
    out = np.full((P, Dp1), -1, dtype=np.int32)
    for p, r in enumerate(rows[:P]):
        out[p, : len(r)] = r
    return out
