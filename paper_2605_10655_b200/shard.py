"""Data-parallel sharding of the path over GPUs: weight blocks are independent, so each rank
takes a contiguous range of blocks; the only quantity that couples ranks is grad_codebook, a
sum over all blocks, which is all-reduced (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Tuple


def block_range(num_blocks: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [start, stop) of the blocks owned by `rank`; sizes differ by at most one."""
    if not (0 <= rank < world) or num_blocks < 0:
        raise ValueError("bad rank/world/num_blocks")
    base, rem = divmod(num_blocks, world)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)


def allreduce_grad_codebook(grad_codebook, group=None):
    """Sum the per-rank partial codebook gradients in place (no-op without a process group)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(grad_codebook, op=dist.ReduceOp.SUM, group=group)
    return grad_codebook
