"""Multi-GPU plumbing: the path shards over independent (batch, layer, KV head) units and
needs no exchange of data, so all that is shared between ranks is a barrier and the
maximum of a timing.  Backend-agnostic (NCCL on GPUs, gloo in the CPU tests)."""
import os

import torch
import torch.distributed as dist


def init(backend, device=None):
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_* (torchrun's variables).
    Returns (rank, world)."""
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, world


def shard_range(n, world, rank):
    """Contiguous share [lo, hi) of n independent items for `rank`; sizes differ by at most one."""
    base, extra = divmod(n, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(x, device="cpu"):
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()
