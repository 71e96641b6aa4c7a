"""Multi-GPU plumbing: one process per GPU, no data-path collective.

Every (batch, head) pair is an independent attention problem (Section 3.1 defines the
method per query row; key and value gradients sum only within a head), so the path shards
over (batch, head) with nothing to exchange.  The only cross-rank traffic is the timing
reduction (maximum over ranks) and barriers around the timed region.
"""
import os

import torch
import torch.distributed as dist


def shard_heads(total_heads: int, world: int, rank: int) -> range:
    """Contiguous, balanced split of the flat (batch*H + head) index range across ranks."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(total_heads, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def init_process_group_from_env(gpus: int, backend: str = "nccl"):
    """Returns (world, rank, local_rank); joins the process group when launched with several ranks."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    if gpus != world and rank == 0 and world > 1:
        raise RuntimeError(f"--gpus {gpus} but WORLD_SIZE={world}")
    return world, rank, local_rank


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Maximum of a per-rank scalar (device timings are reported as the slowest rank's)."""
    if world <= 1 or not dist.is_initialized():
        return float(value)
    if device is None:
        device = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
