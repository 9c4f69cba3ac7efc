"""Multi-GPU plumbing.  The verification step has no data-path exchange
between sequences, so N GPUs run N independent shards of the batch
("prompt_id mod world_size" sharding of Section 4.4) and only timing and
counters cross ranks."""
import os

import torch
import torch.distributed as dist


def init_from_env(backend=None):
    """Join the process group torchrun describes (RANK / WORLD_SIZE / MASTER_*).
    Returns (rank, world_size, local_rank); a plain `python` run is (0, 1, 0)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def shard_sequences(n_sequences, rank, world):
    """Indices of the sequences rank `rank` owns: i with i mod world == rank."""
    return list(range(rank, n_sequences, world))


def _reduce(value, op, device):
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value, device="cpu"):
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value, device="cpu"):
    return _reduce(value, dist.ReduceOp.SUM, device)


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# ---------------------------------------------------------------------------
# Context split: one long prefix spread over the GPUs of a group (Section 6, "Limitations and future work":
# longer-context workloads, multi-device serving).  Every member attends to its own key range and keeps
# (out, lse); the partials are all-gathered into local memory and merged by tree_merge_partials.  No kernel
# reads another GPU's memory.
# ---------------------------------------------------------------------------
def split_prefix(prefix_len, rank, world):
    """Key range [lo, hi) of the committed prefix that member `rank` of a `world`-way context split holds,
    per sequence: lo = floor(S * rank / world), hi = floor(S * (rank + 1) / world).  The ranges of all
    members tile [0, S) without gaps or overlap.  Works on tensors and on plain integers."""
    return (prefix_len * rank) // world, (prefix_len * (rank + 1)) // world


def gather_partials(out, lse, group=None):
    """All-gather the members' (out, lse) into [R, ...] tensors in local memory (R = group size; a process
    outside any group gets R = 1).  The outputs travel as raw bytes, which every backend can move."""
    if not (dist.is_available() and dist.is_initialized()):
        return out.unsqueeze(0).contiguous(), lse.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    o_bits = out.contiguous().view(torch.uint8)
    o_list = [torch.empty_like(o_bits) for _ in range(world)]
    l_list = [torch.empty_like(lse) for _ in range(world)]
    dist.all_gather(o_list, o_bits, group=group)
    dist.all_gather(l_list, lse.contiguous(), group=group)
    return torch.stack(o_list).view(out.dtype), torch.stack(l_list)


def context_split_attention(q, k_cache_local, v_cache_local, k_tree, v_tree, local_prefix_len, n_nodes, anc_bits,
                            scale, workspace, status, owns_tree, group=None, stream=None):
    """tree_verify_attn over a prefix that is split across the members of `group`.

    k_cache_local / v_cache_local hold this member's key range (rows [0, local_prefix_len) of its own
    cache); q, the tree's K/V, n_nodes and anc_bits are the same on every member.  The tree's keys are
    attended to by exactly one member (`owns_tree`); the others run with all-zero ancestor words, so
    their rows see prefix keys only.  Returns (out[B,Nmax,Hq,d] bf16, lse[B,Hq,Nmax] fp32), identical
    on every member."""
    from . import binding as tv
    B, Nmax, Hq, d = q.shape
    bits = anc_bits if owns_tree else torch.zeros_like(anc_bits)
    out_local = torch.empty(B, Nmax, Hq, d, dtype=torch.bfloat16, device=q.device)
    lse_local = torch.empty(B, Hq, Nmax, dtype=torch.float32, device=q.device)
    tv.tree_verify_attn(q, k_cache_local, v_cache_local, k_tree, v_tree, local_prefix_len, n_nodes, bits, scale,
                        out_local, workspace, status, lse=lse_local, stream=stream)
    if stream is not None:
        stream.synchronize()          # the collective below runs on the backend's own stream
    o_parts, lse_parts = gather_partials(out_local, lse_local, group)
    out = torch.empty_like(out_local)
    lse = torch.empty_like(lse_local)
    tv.tree_merge_partials(o_parts, lse_parts, out, lse, stream=stream)
    return out, lse
