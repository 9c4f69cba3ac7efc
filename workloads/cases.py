"""Seeded tensors for one verification step (inputs only, no method arithmetic).

``make_case`` returns torch tensors on the requested device; bf16 data are
``torch.bfloat16``.  ``bf16_bits`` gives the raw uint16 patterns as numpy for
consumers that decode bf16 themselves.
"""
import numpy as np
import torch

from .configs import VerifyConfig
from .trees import (random_parent_tree, topk_expansion_tree, spine_tree, covering_chains_tree, leaf_paths, capped_paths,
                    rows_to_retrieve)

PLANT_LOGIT = 16.0  # far above any N(0,1) draw that survives bf16 rounding


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns of a bf16 tensor as a uint16 numpy array (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 exactly (bf16 is the top half of fp32)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def randn_bf16(shape, std, gen, device, chunk_elems=1 << 26):
    """N(0, std) rounded to bf16, drawn in chunks so that no fp32 temporary of
    the full size is ever held."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        tmp = torch.randn(e - s, generator=gen, device=device, dtype=torch.float32)
        flat[s:e] = (tmp * std).to(torch.bfloat16)
    return out


def _draw_tree(cfg: VerifyConfig, n, rng):
    if n == 1:
        return np.array([-1], dtype=np.int32)
    if n < cfg.N:      # a ragged (smaller) tree: uniform parents, depth bound scaled to its size
        if cfg.tree == "spine":
            return spine_tree(n, min(cfg.D, max(1, (n - 1) // 2)), rng)
        return random_parent_tree(n, min(cfg.D, max(1, (n - 1) // 2)), rng)
    if cfg.tree == "spine":
        return spine_tree(n, min(cfg.D, n - 1), rng)
    if cfg.tree == "chains":         # rows cover every node: P chains from the root
        return covering_chains_tree(n, cfg.P if cfg.P > 0 else -(-(n - 1) // cfg.D), cfg.D, rng)
    if cfg.tree == "uniform":
        return random_parent_tree(n, min(cfg.D, n - 1), rng)
    return topk_expansion_tree(n, cfg.D, cfg.topk, rng)


def make_case(cfg: VerifyConfig, seed: int, device="cpu", ragged_nodes=False,
              with_cache=True, with_logits=True):
    """Draw one step's inputs.

    Returns a dict with (all on ``device``):
      parent[B,N] i32, n_nodes[B] i32, tokens[B,N] i32, retrieve[B,P,D+1] i32,
      prefix_len[B] i32, q[L,B,N,Hq,d], k_tree/v_tree[L,B,N,Hkv,d],
      k_cache/v_cache[L,B,Hkv,Scap,d], logits[B,N,V] (if V>0), and the plan of
      the planted path: plant_row[B], plant_depth[B] (host numpy).
    """
    rng = np.random.default_rng(seed)
    B, N, D = cfg.B, cfg.N, cfg.D
    V = cfg.V if cfg.V > 0 else 32000
    P = cfg.P if cfg.P > 0 else N
    parent = np.zeros((B, N), dtype=np.int32)          # pad fill: parent 0 (device-defined)
    n_nodes = np.full(B, N, dtype=np.int32)
    tokens = rng.integers(0, V, size=(B, N), dtype=np.int64).astype(np.int32)
    retrieve = np.full((B, P, D + 1), -1, dtype=np.int32)
    n_paths = np.zeros(B, dtype=np.int32)
    plant_row = np.zeros(B, dtype=np.int32)
    plant_depth = np.zeros(B, dtype=np.int32)
    plant_edges = []                                   # (b, node_prev, token)
    for b in range(B):
        n = N
        if ragged_nodes and b > 0:
            n = int(rng.integers(1, N + 1))
        n_nodes[b] = n
        par = _draw_tree(cfg, n, rng)
        parent[b, :n] = par
        rows = leaf_paths(par)
        planted = None
        if cfg.plant != "none":
            deepest = max(len(r) for r in rows)
            planted = next(r for r in rows if len(r) == deepest)
        if cfg.P > 0:
            rows = capped_paths(par, cfg.P, None if planted is None else planted[-1])
        retrieve[b] = rows_to_retrieve(rows, P, D + 1)
        n_paths[b] = min(len(rows), P)
        if planted is not None:
            if cfg.plant == "full":
                a = len(planted) - 1
            else:  # geometric on {0,1,..}, success probability 0.18, capped
                a = min(len(planted) - 1, int(rng.geometric(0.18)) - 1)
            plant_row[b] = next(i for i, r in enumerate(rows) if r[-1] == planted[-1])
            plant_depth[b] = a
            for j in range(1, a + 1):
                plant_edges.append((b, planted[j - 1], int(tokens[b, planted[j]])))
    prefix_len = rng.integers(cfg.S_lo, cfg.S_hi + 1, size=B, dtype=np.int64).astype(np.int32)

    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed) * 7919 + 17)
    dev = torch.device(device)
    L, Hq, Hkv, d = cfg.L, cfg.Hq, cfg.Hkv, cfg.d
    case = {
        "cfg": cfg, "seed": seed,
        "parent": torch.from_numpy(parent).to(dev),
        "n_nodes": torch.from_numpy(n_nodes).to(dev),
        "tokens": torch.from_numpy(tokens).to(dev),
        "retrieve": torch.from_numpy(retrieve).to(dev),
        "n_paths": n_paths,
        "prefix_len": torch.from_numpy(prefix_len).to(dev),
        "plant_row": plant_row, "plant_depth": plant_depth,
        "q": randn_bf16((L, B, N, Hq, d), cfg.std, gen, dev),
        "k_tree": randn_bf16((L, B, N, Hkv, d), cfg.std, gen, dev),
        "v_tree": randn_bf16((L, B, N, Hkv, d), cfg.std, gen, dev),
    }
    if with_cache:
        case["k_cache"] = randn_bf16((L, B, Hkv, cfg.Scap, d), cfg.std, gen, dev)
        case["v_cache"] = randn_bf16((L, B, Hkv, cfg.Scap, d), cfg.std, gen, dev)
    if cfg.V > 0 and with_logits:
        logits = randn_bf16((B, N, cfg.V), 1.0, gen, dev)
        for (b, node, tok) in plant_edges:
            logits[b, node, tok] = PLANT_LOGIT
        case["logits"] = logits
    return case


def case_to_numpy(case):
    """Host copy of a case: bf16 tensors become uint16 bit patterns, integer
    tensors numpy arrays; everything else is passed through."""
    out = {}
    for k, v in case.items():
        if isinstance(v, torch.Tensor):
            out[k] = bf16_bits(v) if v.dtype == torch.bfloat16 else v.detach().cpu().numpy()
        else:
            out[k] = v
    return out
