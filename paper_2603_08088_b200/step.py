"""Device buffers for one verification step and the call sequence of a step.

Only allocation and call ordering live here (tensorise + mask, attention per
layer, gather + accept, commit - the order of Section 3); every computation is
inside the library calls.
"""
import torch

from . import binding as tv


class StepBuffers:
    """Outputs and scratch of a step for fixed dimensions, allocated once."""

    def __init__(self, L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1, device="cuda", want_dense=False,
                 want_lse=False, want_gather=False):
        i32 = dict(dtype=torch.int32, device=device)
        W = (Nmax + 31) // 32
        self.dims = (L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1)
        self.anc_bits = torch.zeros(B, Nmax, W, **i32)
        self.status = torch.zeros(B, **i32)
        self.depth = torch.zeros(B, Nmax, **i32)
        self.anc_table = torch.zeros(B, Dp1, Nmax, **i32)
        self.retrieve = torch.full((B, max(P, 1), Dp1), -1, **i32)
        self.n_paths = torch.zeros(B, **i32)
        self.dense = torch.zeros(B, 1, Nmax, Nmax, dtype=torch.uint8, device=device) if want_dense else None
        self.out = torch.zeros(L, B, Nmax, Hq, d, dtype=torch.bfloat16, device=device)
        self.lse = torch.zeros(L, B, Hq, Nmax, dtype=torch.float32, device=device) if want_lse else None
        self.attn_ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, Nmax, Hq, Hkv, d, Scap)),
                                   dtype=torch.uint8, device=device)
        if V > 0:
            self.accept_ws = torch.zeros(max(16, tv.tv_accept_workspace_bytes(B, Nmax, V)),
                                         dtype=torch.uint8, device=device)
            self.argmax_tok = torch.zeros(B, Nmax, **i32)
            self.accept_len = torch.zeros(B, **i32)
            self.best_path = torch.zeros(B, **i32)
            self.accepted_nodes = torch.zeros(B, Dp1, **i32)
            self.next_token = torch.zeros(B, **i32)
            self.safe_idx = torch.zeros(B, max(P, 1), Dp1, **i32) if want_gather else None
            self.candidates = torch.zeros(B, max(P, 1), Dp1, **i32) if want_gather else None


def verify_step(case, buf: StepBuffers, scale, retrieve=None, commit=True, stream=None, in_cache=False):
    """Enqueue one whole step on ``stream`` (default: torch's current stream).

    ``case`` holds device tensors parent, n_nodes, tokens, prefix_len, q, k_tree, v_tree
    [L,...], k_cache, v_cache [L,...] and logits (optional).  ``retrieve`` overrides the
    candidate rows; by default the rows tree_build_mask emits are used.  ``in_cache``: the tree's K/V are
    rows prefix_len[b] + node of the caches (k_tree / v_tree are not read) and the commit reorders in place.
    """
    L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1 = buf.dims
    own_rows = retrieve is None
    tv.tree_build_mask(case["parent"], case["n_nodes"], Dp1 - 1, buf.retrieve.shape[1], buf.anc_bits, buf.status,
                       dense_mask=buf.dense, depth=buf.depth, anc_table=buf.anc_table,
                       retrieve_indices=buf.retrieve if own_rows else None,
                       n_paths=buf.n_paths, stream=stream)
    # all layers in one call; the mask kernel in front leaves prefix_len and the cache alone, so the first layer
    # may start under it as well
    tv.tree_verify_attn_layers(case["q"], case["k_cache"], case["v_cache"],
                               None if in_cache else case["k_tree"], None if in_cache else case["v_tree"],
                               case["prefix_len"], case["n_nodes"], buf.anc_bits, scale, buf.out, buf.attn_ws,
                               buf.status, lse=buf.lse, flags=tv.TV_ATTN_STABLE_INPUTS, stream=stream)
    if V > 0 and "logits" in case:
        rows = buf.retrieve if own_rows else retrieve
        tv.tree_accept(case["logits"], case["tokens"], rows, case["n_nodes"], buf.argmax_tok, buf.accept_len,
                       buf.best_path, buf.accepted_nodes, buf.next_token, buf.accept_ws, buf.status,
                       safe_idx=buf.safe_idx, candidates=buf.candidates, stream=stream)
        if commit and in_cache:
            tv.kv_commit_inplace(case["k_cache"], case["v_cache"], buf.accepted_nodes, buf.accept_len,
                                 case["prefix_len"], Nmax, buf.status, stream=stream)
        elif commit:
            tv.kv_commit(case["k_cache"], case["v_cache"], case["k_tree"], case["v_tree"], buf.accepted_nodes,
                         buf.accept_len, case["prefix_len"], buf.status, stream=stream)
