"""Host-side partitioning of the four operations across GPUs (one process per GPU).

Every forward operation of the library decomposes into independent units -- rows of A/D for a GEMM,
batch entries, whole groups, images of a convolution -- so a multi-GPU run needs no exchange
step on the data path: each rank runs the single-GPU kernel on its shard.  The partition functions
are pure integer arithmetic (no tensors, no CUDA) so they can be tested with CPU process groups.
The one operation with a real exchange step is the data-parallel weight gradient: its sum runs over
the images, so the ranks' partial dW are added with an all-reduce (``reduce_weight_gradient``).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def split_range(total: int, world: int, rank: int, multiple: int = 1) -> Tuple[int, int]:
    """Contiguous [begin, end) of `total` units for `rank`; all cuts but the last fall on a multiple
    of `multiple` (e.g. the 128-row tile height), sizes differ by at most one such block."""
    if world < 1 or not 0 <= rank < world or total < 0 or multiple < 1:
        raise ValueError("bad partition request")
    blocks = -(-total // multiple)
    base, extra = divmod(blocks, world)
    begin_b = rank * base + min(rank, extra)
    end_b = begin_b + base + (1 if rank < extra else 0)
    return min(begin_b * multiple, total), min(end_b * multiple, total)


def gemm_rows(M: int, world: int, rank: int, tile_m: int = 128) -> Tuple[int, int]:
    """Rows of A and D this rank computes (B is replicated)."""
    return split_range(M, world, rank, tile_m)


def batch_entries(batch: int, world: int, rank: int) -> Tuple[int, int]:
    return split_range(batch, world, rank)


def conv_images(N: int, world: int, rank: int) -> Tuple[int, int]:
    """Images this rank convolves (the filter is replicated)."""
    return split_range(N, world, rank)


def assign_groups(Ms: Sequence[int], world: int) -> List[List[int]]:
    """Whole groups per rank, balanced by row count: largest group first onto the lightest rank."""
    if world < 1:
        raise ValueError("world must be >= 1")
    loads = [0] * world
    owned: List[List[int]] = [[] for _ in range(world)]
    for g in sorted(range(len(Ms)), key=lambda i: (-Ms[i], i)):
        r = min(range(world), key=lambda i: (loads[i], i))
        owned[r].append(g)
        loads[r] += Ms[g]
    for lst in owned:
        lst.sort()
    return owned


def reduce_weight_gradient(dW, group=None):
    """Data-parallel ``conv2d_wgrad``: every rank has summed over its own images (``conv_images``); the filter
    gradient is the sum over all images, i.e. an all-reduce of the ranks' dW (NCCL on GPUs, gloo on CPU), in place."""
    import torch.distributed as dist
    dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
    return dW
