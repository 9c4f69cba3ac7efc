"""CPU oracle for the tree-verification step (TEST INFRASTRUCTURE, not product).

Plain, slow, fp64 numpy restatement of what one teacher tree-verification
step of EAGLE-3-style tree speculative decoding computes, written from the
paper's problem statement.  It shares no code with the CUDA library and must
only be imported by tests, the smoke check and the bench's CPU-baseline legs.
Every function cites the passage it follows.  Nothing here is blocked, fused
or reordered beyond the definitions; a library matmul / exp / max serves as a
step where the definition is a sum, an exponential or a maximum.

Conventions (same index algebra as Section 3.2 with N = M + 1 rows):
  * node 0 is the root (the last sampled token, row 0 of the paper's
    (M+1)-row tensors); ``parent[0] = -1`` is the only sentinel and is
    remapped to 0 before any gather (dummy-root indexing);
  * ``valid[i] = i < n_nodes``; padded slots carry device-defined fill
    (parent 0, depth 0) and never influence active outputs;
  * bf16 data arrive as uint16 bit patterns and are decoded here.

Parity status: every function below is pinned by tests/test_oracle_pins.py
(brute force, closed forms, library routines, special trees); none is
"parity unpinned".
"""
import numpy as np

# status bits reported per sequence
ST_BAD_TREE = 1          # a structural invariant of Section 3.2 failed
ST_BAD_INDEX = 2         # a path / node index outside [-1, n_nodes)
ST_CAPACITY = 4          # commit would run past the cache capacity
ST_TIMEOUT = 8           # (device only) a bounded wait expired
ST_PATHS_TRUNCATED = 16  # more leaves than path rows; non-fatal
ST_FATAL = ST_BAD_TREE | ST_BAD_INDEX | ST_CAPACITY | ST_TIMEOUT


def decode_bf16(bits):
    """bf16 bit patterns -> float64, exactly (bf16 is the upper half of an fp32)."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ---------------------------------------------------------------------------
# Section 3.2: tensorisation (dummy-root remap, depth, ancestor table, invariants)
# ---------------------------------------------------------------------------
def tensorize_one(parent, n, Dcap):
    """One sequence.  Returns (ok, safe_parent, depth, A) with A of shape
    [Dcap+1, Nmax]; on an invariant failure ok is False and the arrays are zero.

    Dummy-root indexing: safe_parent[i] = 0 where parent[i] is the sentinel
    (Section 3.2, "Dummy-root indexing").  Ancestor table: A[0,i] = i,
    A[l+1,i] = safe_parent[A[l,i]] (Section 3.2, "Ancestor tables").
    Invariants (Section 3.2, "Structural invariants"): range, depth
    consistency / acyclicity (parent chain reaches 0 within depth steps),
    validity closure; plus our topological-order reading parent[i] < i and
    the caller's depth bound.
    """
    Nmax = len(parent)
    sp = np.zeros(Nmax, dtype=np.int32)
    depth = np.zeros(Nmax, dtype=np.int32)
    A = np.zeros((Dcap + 1, Nmax), dtype=np.int32)
    zero = (False, np.zeros_like(sp), np.zeros_like(depth), np.zeros_like(A))
    if n < 1 or n > Nmax:
        return zero
    if parent[0] != -1:
        return zero
    for i in range(1, n):
        p = int(parent[i])
        if p < 0 or p >= n:          # range
            return zero
        if p >= i:                   # topological order (our reading)
            return zero
        sp[i] = p
    # padded slots: device-defined fill, parent 0 / depth 0, whatever the input holds
    for i in range(1, n):
        # depth by a capped parent walk: steps until row 0 is reached
        cur, steps = i, 0
        while cur != 0 and steps <= n:
            cur = int(sp[cur])
            steps += 1
        if cur != 0:                 # acyclicity
            return zero
        depth[i] = steps
    for i in range(1, n):
        if not depth[sp[i]] < depth[i]:   # depth consistency
            return zero
        if depth[i] > Dcap:
            return zero
        if not sp[i] < n:                 # validity closure (valid => parent valid)
            return zero
    for i in range(Nmax):
        A[0, i] = i
    for l in range(Dcap):
        for i in range(Nmax):
            A[l + 1, i] = sp[A[l, i]]
    for i in range(1, n):
        if A[depth[i], i] != 0:
            return zero
    return True, sp, depth, A


def build_mask(parent, n_nodes, Dcap, Pcap, emit_paths=True):
    """Tree tensorisation + mask for a batch (Sections 2.4, 3.2, 3.3).

    vis[b,i,j] = valid[i] and valid[j] and (exists l in [0,Dcap]: A[l,i] == j)
    is the ancestor-or-self predicate of Section 3.3 combined with the
    no-leak padding rule.  Returns a dict:
      anc_bits[B,Nmax,W] u32 (bit j%32 of word j//32 of row i), dense[B,1,Nmax,Nmax] u8,
      depth[B,Nmax], anc_table[B,Dcap+1,Nmax], retrieve[B,Pcap,Dcap+1] (-1 padded),
      n_paths[B], status[B].
    Candidate-path rows: one per leaf, leaves in increasing node id, root
    first, -1 after the leaf.  With emit_paths=False no rows are written
    (they stay -1), n_paths is the leaf count and nothing can be truncated.
    """
    parent = np.asarray(parent)
    B, Nmax = parent.shape
    W = (Nmax + 31) // 32
    out = {
        "anc_bits": np.zeros((B, Nmax, W), dtype=np.uint32),
        "dense": np.zeros((B, 1, Nmax, Nmax), dtype=np.uint8),
        "depth": np.zeros((B, Nmax), dtype=np.int32),
        "anc_table": np.zeros((B, Dcap + 1, Nmax), dtype=np.int32),
        "retrieve": np.full((B, Pcap, Dcap + 1), -1, dtype=np.int32),
        "n_paths": np.zeros(B, dtype=np.int32),
        "status": np.zeros(B, dtype=np.int32),
    }
    for b in range(B):
        n = int(n_nodes[b])
        ok, sp, depth, A = tensorize_one(parent[b], n, Dcap)
        if not ok:
            out["status"][b] = ST_BAD_TREE
            continue
        out["depth"][b] = depth
        out["anc_table"][b] = A
        for i in range(n):
            for j in range(n):
                seen = False
                for l in range(Dcap + 1):
                    if A[l, i] == j:
                        seen = True
                if seen:
                    out["dense"][b, 0, i, j] = 1
                    out["anc_bits"][b, i, j // 32] |= np.uint32(1) << np.uint32(j % 32)
        # root-to-leaf rows
        has_child = np.zeros(n, dtype=bool)
        for i in range(1, n):
            has_child[sp[i]] = True
        row = 0
        for leaf in range(n):
            if has_child[leaf]:
                continue
            if not emit_paths:
                row += 1
                continue
            if row >= Pcap:
                out["status"][b] |= ST_PATHS_TRUNCATED
                break
            dl = int(depth[leaf])
            for l in range(dl + 1):
                out["retrieve"][b, row, dl - l] = A[l, leaf]
            row += 1
        out["n_paths"][b] = row
    return out


# ---------------------------------------------------------------------------
# Sections 2.3, 3.3: tree attention (the attention sub-step of TeacherTreeEval)
# ---------------------------------------------------------------------------
def tree_attention(q_bits, k_cache_bits, v_cache_bits, k_tree_bits, v_tree_bits,
                   prefix_len, n_nodes, vis, scale):
    """Every valid node i, query head h (KV head h // G) attends the committed
    prefix rows [0, S_b) and the tree keys j with vis[b,i,j] (context
    correctness, Section 3.3): softmax with max subtraction over
    scale * <q, k>, times V.  Shapes: q[B,Nmax,Hq,d], caches[B,Hkv,Scap,d],
    tree K/V[B,Nmax,Hkv,d], vis[B,Nmax,Nmax] (0/1).
    Returns out[B,Nmax,Hq,d] f64 and lse[B,Hq,Nmax] f64; rows without any
    visible key (padded rows) give zeros and -inf.
    """
    q = decode_bf16(q_bits)
    B, Nmax, Hq, d = q.shape
    Hkv = k_cache_bits.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Nmax, Hq, d), dtype=np.float64)
    lse = np.full((B, Hq, Nmax), -np.inf, dtype=np.float64)
    for b in range(B):
        S = int(prefix_len[b])
        n = int(n_nodes[b])
        for h in range(Hq):
            hk = h // G
            keys = np.concatenate([decode_bf16(k_cache_bits[b, hk, :S]),
                                   decode_bf16(k_tree_bits[b, :, hk])], axis=0)
            vals = np.concatenate([decode_bf16(v_cache_bits[b, hk, :S]),
                                   decode_bf16(v_tree_bits[b, :, hk])], axis=0)
            x = scale * (q[b, :, h, :] @ keys.T)                    # [Nmax, S+Nmax]
            see = np.zeros((Nmax, S + Nmax), dtype=bool)
            see[:n, :S] = True
            see[:, S:] = np.asarray(vis[b], dtype=bool)
            see[n:, :] = False
            for i in range(Nmax):
                cols = np.flatnonzero(see[i])
                if cols.size == 0:
                    continue
                xi = x[i, cols]
                m = xi.max()
                p = np.exp(xi - m)
                l = p.sum()
                out[b, i, h, :] = (p / l) @ vals[cols]
                lse[b, h, i] = m + np.log(l)
    return out, lse


def merge_partials(o_parts, lse_parts):
    """Attention over a key set split in R disjoint ranges, from the per-range results (the context split
    that longer-context, multi-device serving needs; Section 6, "Limitations and future work"; the
    attention itself is Section 2.4).  For one query row, range r gives O_r = softmax over its own keys
    times V and lse_r = log of the sum of exp(score) over its keys; over the union the softmax weights are
    exp(score) / sum_r exp(lse_r), so  O = sum_r exp(lse_r) O_r / sum_r exp(lse_r)  and
    lse = log sum_r exp(lse_r)  (evaluated with the maximum subtracted).  A range without visible keys has
    lse_r = -inf and weight 0; a row without any key gives zeros and -inf.
    o_parts[R,B,Nmax,Hq,d], lse_parts[R,B,Hq,Nmax] -> out[B,Nmax,Hq,d] f64, lse[B,Hq,Nmax] f64."""
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    R, B, Nmax, Hq, d = o_parts.shape
    out = np.zeros((B, Nmax, Hq, d), dtype=np.float64)
    lse = np.full((B, Hq, Nmax), -np.inf, dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            for i in range(Nmax):
                l = lse_parts[:, b, h, i]
                m = l.max()
                if m == -np.inf:
                    continue
                w = np.exp(l - m)                      # exp(-inf) = 0 for empty ranges
                tot = w.sum()
                acc = np.zeros(d, dtype=np.float64)
                for r in range(R):
                    if w[r] > 0.0:                     # an empty range may carry anything in O_r
                        acc += w[r] * o_parts[r, b, i, h, :]
                out[b, i, h, :] = acc / tot
                lse[b, h, i] = m + np.log(tot)
    return out, lse


# ---------------------------------------------------------------------------
# Sections 2.5, 3.2: accelerator-safe path gather
# ---------------------------------------------------------------------------
def safe_gather(retrieve, tokens, n_nodes):
    """Sentinel -> dummy index 0 *before* the gather, guarded by a validity
    flag (Section 2.5; Section 3.2 "Dummy-root indexing", "Padding and batch
    semantics").  retrieve[B,P,Dp1], tokens[B,Nmax].
    Returns safe_idx, cand (tokens[safe_idx]), ok, status[B].
    """
    retrieve = np.asarray(retrieve)
    B, P, Dp1 = retrieve.shape
    safe = np.zeros_like(retrieve)
    cand = np.zeros_like(retrieve)
    ok = np.zeros(retrieve.shape, dtype=bool)
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = int(n_nodes[b])
        for p in range(P):
            for j in range(Dp1):
                r = int(retrieve[b, p, j])
                good = 0 <= r < n
                if r < -1 or r >= n:
                    status[b] |= ST_BAD_INDEX
                s = r if good else 0
                assert 0 <= s < tokens.shape[1]      # every dereferenced index is in range
                safe[b, p, j] = s
                ok[b, p, j] = good
                cand[b, p, j] = tokens[b, s]
    return safe, cand, ok, status


# ---------------------------------------------------------------------------
# Section 2.1: greedy teacher choice; Section 2.3: acceptance along one path
# ---------------------------------------------------------------------------
def argmax_rows(logits_bits, n_nodes):
    """am[b,i] = the lowest v with logits[b,i,v] equal to the row maximum
    (greedy selection of Section 2.1, temperature 0 as in Section 5); -1 for
    padded rows.  Comparison is on the decoded float values, so -0.0 == +0.0."""
    B, Nmax, V = logits_bits.shape
    am = np.full((B, Nmax), -1, dtype=np.int32)
    for b in range(B):
        for i in range(int(n_nodes[b])):
            row = decode_bf16(logits_bits[b, i])
            top = row.max()
            am[b, i] = np.flatnonzero(row == top)[0]
    return am


def node_scores(logits_bits, tokens, parent, n_nodes):
    """Teacher score of every node's proposed token (Section 3.3, "Mapping teacher outputs to node
    verification scores"): the logits that predict node k's token are those computed at its parent's
    slot, so score[b,k] = logits[b, parent~[k], tokens[b,k]] with the dummy-root remap of Section 3.2.
    An in-range gather over the vocabulary guarded by valid: the root (already part of the prefix) and
    padded slots give 0; a token outside [0,V) is remapped to 0 before the gather, scores -inf and
    raises BAD_INDEX.  Returns scores[B,Nmax] (float32 values of the bf16 logits) and status[B]."""
    B, Nmax, V = logits_bits.shape
    scores = np.zeros((B, Nmax), dtype=np.float32)
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = int(n_nodes[b])
        for k in range(1, min(n, Nmax)):
            p = int(parent[b, k])
            sp = p if 0 <= p < n else 0
            t = int(tokens[b, k])
            ok = 0 <= t < V
            st = t if ok else 0
            assert 0 <= sp < Nmax and 0 <= st < V          # every dereferenced index is in range
            val = np.float32(decode_bf16(logits_bits[b, sp, st]))
            if ok:
                scores[b, k] = val
            else:
                scores[b, k] = -np.inf
                status[b] |= ST_BAD_INDEX
    return scores, status


def stochastic_accept(logits_bits, tokens, parent, n_nodes, u_node, u_bonus, temperature, Dp1):
    """Sampling-mode acceptance over the tree (Section 2.2: an acceptance rule "rejection sampling
    style ... so that the resulting marginal distribution matches the teacher distribution"; Section
    3.3: the node scores l(k) are what the rule consumes).  The paper prints no formula; this is the
    speculative-sampling rule of the work it cites, for proposals that carry no draft probability
    (q = one-hot on the proposed token), walked down the tree:

      at the current node c (the root first) the teacher distribution is p = softmax(logits[c] / T);
      its children k (parent[k] = c, increasing node id, valid slots only) are tried in turn:
        x = tokens[k]; a token already rejected at this node is skipped;
        accept k iff u_node[k] < p(x) / (1 - mass rejected so far at this node)
        (= min(1, p'/q) with q = 1 and p' the distribution renormalised after the rejections);
        otherwise x is rejected: its mass is removed and the next child is tried;
      an accepted child becomes the current node (at most Dp1 - 1 accepted nodes);
      when no child is accepted, the next token is drawn from p with the rejected tokens removed,
      by inversion of the cumulative sum in vocabulary order at u_bonus.

    The uniforms are inputs: u_node[B,Nmax] (one per node, read when that node is tried) and
    u_bonus[B], all in [0,1).  Returns accept_len, accepted_nodes [B,Dp1] (first A+1 valid, rest 0),
    next_token, status (BAD_INDEX if any valid non-root slot proposes a token outside [0,V); such a
    child is never accepted).  A sequence without nodes returns accept_len 0 and next_token -1.
    T -> 0 gives the greedy rule; every output token is distributed as under plain sampling from the
    teacher (the property the pins check).
    """
    B, Nmax, V = logits_bits.shape
    accept_len = np.zeros(B, dtype=np.int32)
    accepted_nodes = np.zeros((B, Dp1), dtype=np.int32)
    next_token = np.zeros(B, dtype=np.int32)
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = int(min(max(int(n_nodes[b]), 0), Nmax))
        if n == 0:
            next_token[b] = -1
            continue
        if any(not (0 <= int(tokens[b, k]) < V) for k in range(1, n)):
            status[b] |= ST_BAD_INDEX
        c, depth = 0, 0
        while True:
            row = decode_bf16(logits_bits[b, c]).astype(np.float64) / float(temperature)
            e = np.exp(row - row.max())
            rejected = []
            accepted = -1
            if depth < Dp1 - 1:
                for k in range(max(c, 0) + 1, n):
                    pk = int(parent[b, k])
                    if (pk if 0 <= pk < n else 0) != c:
                        continue
                    x = int(tokens[b, k])
                    if not (0 <= x < V):
                        continue
                    if x in rejected:
                        continue
                    kept = e.copy()
                    kept[rejected] = 0.0
                    rem = kept.sum()
                    prob = e[x] / rem if rem > 0 else 0.0
                    if float(u_node[b, k]) < prob:
                        accepted = k
                        break
                    rejected.append(x)
            if accepted < 0:
                kept = e.copy()
                kept[rejected] = 0.0
                cum = np.cumsum(kept)
                target = float(u_bonus[b]) * cum[-1]
                next_token[b] = min(int(np.searchsorted(cum, target, side="right")), V - 1)
                break
            depth += 1
            accepted_nodes[b, depth] = accepted
            c = accepted
        accept_len[b] = depth
    return {"accept_len": accept_len, "accepted_nodes": accepted_nodes, "next_token": next_token, "status": status}


def greedy_accept(retrieve, tokens, n_nodes, am):
    """Longest accepted prefix over all candidate rows (Section 2.3: accepted
    nodes form a single root-to-leaf path prefix; greedy rule, Section 5).

    A draft node on a row is accepted when its token equals the teacher's
    argmax at the previous node of the row and all earlier nodes of the row
    were accepted; remapped (-1) slots never match because of the validity
    guard.  Ties between rows go to the lowest row.
    Returns accept_len[B], best_path[B], accepted_nodes[B,Dp1] (first A+1
    entries, rest 0), next_token[B] (teacher argmax at the last accepted
    node), safe_idx, cand, status.
    """
    safe, cand, ok, status = safe_gather(retrieve, tokens, n_nodes)
    B, P, Dp1 = safe.shape
    accept_len = np.zeros(B, dtype=np.int32)
    best_path = np.zeros(B, dtype=np.int32)
    accepted = np.zeros((B, Dp1), dtype=np.int32)
    next_token = np.zeros(B, dtype=np.int32)
    for b in range(B):
        best_a, best_p = 0, 0
        for p in range(P):
            a = 0
            for j in range(1, Dp1):
                if ok[b, p, j] and ok[b, p, j - 1] and cand[b, p, j] == am[b, safe[b, p, j - 1]]:
                    a = j
                else:
                    break
            if a > best_a:
                best_a, best_p = a, p
        accept_len[b] = best_a
        best_path[b] = best_p
        if P > 0:
            for j in range(best_a + 1):
                accepted[b, j] = safe[b, best_p, j]
        next_token[b] = am[b, accepted[b, best_a]]
    return {"accept_len": accept_len, "best_path": best_path, "accepted_nodes": accepted,
            "next_token": next_token, "safe_idx": safe, "candidates": cand, "ok": ok,
            "status": status}


# ---------------------------------------------------------------------------
# Section 3.1: path-index commit, prefix-sharing fast reorder
# ---------------------------------------------------------------------------
def kv_commit(k_cache, v_cache, k_tree, v_tree, accepted_nodes, accept_len, prefix_len,
              status_in=None):
    """The committed prefix keeps its order and only the accepted segment is
    gathered behind it (Section 3.1, "Prefix-sharing fast reorder"):
    cache[l,b,h,S_b+j,:] = tree[l,b,accepted_nodes[b,j],h,:] for j = 0..A_b,
    then prefix_len[b] += A_b + 1.  Works on copies; all other bytes are
    unchanged.  A sequence whose incoming status is fatal, whose segment
    would pass the capacity or whose node list leaves [0,Nmax) is skipped and
    flagged.  Arrays are raw uint16 (any dtype works: this is a byte copy).
    """
    kc, vc = k_cache.copy(), v_cache.copy()
    L, B, Hkv, Scap, d = kc.shape
    Nmax = k_tree.shape[2]
    Dp1 = accepted_nodes.shape[1]
    new_len = np.array(prefix_len, dtype=np.int32).copy()
    status = np.zeros(B, dtype=np.int32) if status_in is None else np.array(status_in, dtype=np.int32).copy()
    for b in range(B):
        if status[b] & ST_FATAL:
            continue
        S, A = int(prefix_len[b]), int(accept_len[b])
        if A < 0 or A >= Dp1 or any(not (0 <= int(accepted_nodes[b, j]) < Nmax) for j in range(A + 1)):
            status[b] |= ST_BAD_INDEX
            continue
        if S < 0 or S + A + 1 > Scap:
            status[b] |= ST_CAPACITY
            continue
        for l in range(L):
            for h in range(Hkv):
                for j in range(A + 1):
                    node = int(accepted_nodes[b, j])
                    kc[l, b, h, S + j, :] = k_tree[l, b, node, h, :]
                    vc[l, b, h, S + j, :] = v_tree[l, b, node, h, :]
        new_len[b] = S + A + 1
    return kc, vc, new_len, status


def kv_commit_inplace(k_cache, v_cache, accepted_nodes, accept_len, prefix_len, Nmax, status_in=None):
    """Path-index commit as a full reorder (Section 3.1, "Full reordering"),
    for a cache the teacher forward extended in place: node i of the tree sits
    at row S_b + i.  The new committed cache is the gather of the OLD one along
    the sequence axis by path_indices = [0..S_b-1, S_b + accepted_nodes[b,0..A_b]]:
    new[l,b,h,t,:] = old[l,b,h,path_indices[t],:] for t < S_b + A_b + 1.  Rows
    below S_b map to themselves; rows at or past S_b + A_b + 1 are outside the
    new committed length and keep their bytes.  Works on copies.  Skips and
    flags a sequence as kv_commit does; a source row at or past the capacity
    is a capacity error too.
    """
    kc, vc = k_cache.copy(), v_cache.copy()
    L, B, Hkv, Scap, d = kc.shape
    Dp1 = accepted_nodes.shape[1]
    new_len = np.array(prefix_len, dtype=np.int32).copy()
    status = np.zeros(B, dtype=np.int32) if status_in is None else np.array(status_in, dtype=np.int32).copy()
    for b in range(B):
        if status[b] & ST_FATAL:
            continue
        S, A = int(prefix_len[b]), int(accept_len[b])
        if A < 0 or A >= Dp1 or any(not (0 <= int(accepted_nodes[b, j]) < Nmax) for j in range(A + 1)):
            status[b] |= ST_BAD_INDEX
            continue
        if S < 0 or S + A + 1 > Scap or any(S + int(accepted_nodes[b, j]) >= Scap for j in range(A + 1)):
            status[b] |= ST_CAPACITY
            continue
        path_indices = list(range(S)) + [S + int(accepted_nodes[b, j]) for j in range(A + 1)]
        T = len(path_indices)
        kc[:, b, :, :T, :] = k_cache[:, b][:, :, path_indices, :]      # gather from the old cache
        vc[:, b, :, :T, :] = v_cache[:, b][:, :, path_indices, :]
        new_len[b] = T
    return kc, vc, new_len, status


# ---------------------------------------------------------------------------
# Paged cache ("backend-specific layouts", Section 3.1): the same committed
# rows, stored in pages of 128 rows named by a block table
# ---------------------------------------------------------------------------
PAGE_ROWS = 128


def paged_to_contiguous(pages, block_table):
    """pages [n_pages,Hkv,128,d], block_table [B,max_blocks] -> the cache as
    [B,Hkv,128*max_blocks,d]: row s of sequence b is row s % 128 of page
    block_table[b, s // 128].  Every table entry must name a page."""
    n_pages = pages.shape[0]
    bt = np.asarray(block_table)
    assert ((0 <= bt) & (bt < n_pages)).all()
    g = pages[bt]                                   # [B, max_blocks, Hkv, 128, d]
    B, nb, Hkv, R, d = g.shape
    return g.transpose(0, 2, 1, 3, 4).reshape(B, Hkv, nb * R, d)


def kv_commit_paged(k_pages, v_pages, block_table, k_tree, v_tree, accepted_nodes, accept_len, prefix_len,
                    status_in=None):
    """kv_commit on a paged cache: row S_b + j of sequence b lives in page
    block_table[b, (S_b+j) // 128] at row (S_b+j) % 128.  pages are
    [L,n_pages,Hkv,128,d]; works on copies.  The capacity is 128 * max_blocks;
    a page id outside [0, n_pages) under the accepted segment is an index
    error and skips the sequence."""
    kp, vp = k_pages.copy(), v_pages.copy()
    L, n_pages, Hkv, R, d = kp.shape
    B, max_blocks = block_table.shape
    Nmax = k_tree.shape[2]
    Dp1 = accepted_nodes.shape[1]
    new_len = np.array(prefix_len, dtype=np.int32).copy()
    status = np.zeros(B, dtype=np.int32) if status_in is None else np.array(status_in, dtype=np.int32).copy()
    for b in range(B):
        if status[b] & ST_FATAL:
            continue
        S, A = int(prefix_len[b]), int(accept_len[b])
        if A < 0 or A >= Dp1 or any(not (0 <= int(accepted_nodes[b, j]) < Nmax) for j in range(A + 1)):
            status[b] |= ST_BAD_INDEX
            continue
        if S < 0 or S + A + 1 > R * max_blocks:
            status[b] |= ST_CAPACITY
            continue
        if any(not (0 <= int(block_table[b, t]) < n_pages) for t in range(S // R, (S + A) // R + 1)):
            status[b] |= ST_BAD_INDEX
            continue
        for j in range(A + 1):
            row, node = S + j, int(accepted_nodes[b, j])
            pg = int(block_table[b, row // R])
            kp[:, pg, :, row % R, :] = k_tree[:, b, node, :, :]
            vp[:, pg, :, row % R, :] = v_tree[:, b, node, :, :]
        new_len[b] = S + A + 1
    return kp, vp, new_len, status


def verify_step(case_np, scale, Dcap=None, Pcap=None, use_given_retrieve=True):
    """One whole step in the paper's order: tensorise + mask, attention per
    layer, safe gather + argmax + accept, commit (Section 3 call order)."""
    parent, n_nodes = case_np["parent"], case_np["n_nodes"]
    Dp1 = case_np["retrieve"].shape[2]
    mk = build_mask(parent, n_nodes, Dp1 - 1 if Dcap is None else Dcap,
                    case_np["retrieve"].shape[1] if Pcap is None else Pcap,
                    emit_paths=not (use_given_retrieve and "logits" in case_np))
    L = case_np["q"].shape[0]
    outs, lses = [], []
    for l in range(L):
        o, s = tree_attention(case_np["q"][l], case_np["k_cache"][l], case_np["v_cache"][l],
                              case_np["k_tree"][l], case_np["v_tree"][l],
                              case_np["prefix_len"], n_nodes, mk["dense"][:, 0], scale)
        outs.append(o)
        lses.append(s)
    res = {"mask": mk, "out": np.stack(outs), "lse": np.stack(lses)}
    if "logits" in case_np:
        am = argmax_rows(case_np["logits"], n_nodes)
        retrieve = case_np["retrieve"] if use_given_retrieve else mk["retrieve"]
        acc = greedy_accept(retrieve, case_np["tokens"], n_nodes, am)
        status = mk["status"] | acc["status"]
        kc, vc, new_len, status = kv_commit(case_np["k_cache"], case_np["v_cache"],
                                            case_np["k_tree"], case_np["v_tree"],
                                            acc["accepted_nodes"], acc["accept_len"],
                                            case_np["prefix_len"], status)
        res.update({"argmax": am, "accept": acc, "k_cache": kc, "v_cache": vc,
                    "prefix_len": new_len, "status": status})
    return res
