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
