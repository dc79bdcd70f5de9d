"""Image sharding for several GPUs: one process per GPU, no exchange on the data path.

The Monte-Carlo loop of one image never needs another image's data, so CERTIFY over a set of images
partitions by image: rank r certifies a contiguous block of images with their global image ids (the id
selects the random stream, so results do not depend on the number of ranks) and the per-image results
are gathered once at the end.  `certify_fn(images_block, first_image_id)` is the per-rank worker -- on a
GPU machine `Model.certify_batch`; any callable with the same contract works.
"""
from __future__ import annotations

import numpy as np


def image_block(rank: int, world: int, n_images: int):
    """[begin, end) of the images rank `rank` of `world` certifies (blocks differ by at most one image)."""
    base, extra = divmod(n_images, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def certify_sharded(certify_fn, images: np.ndarray, image_id0: int = 0, group=None):
    """Certify images[begin:end) on this rank and return the results of ALL images on every rank.

    certify_fn(block, first_id) -> (classes[n], radii[n], counts0[n, C], counts[n, C])
    """
    import torch.distributed as dist
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    begin, end = image_block(rank, world, len(images))
    mine = certify_fn(images[begin:end], image_id0 + begin) if end > begin else None
    if world == 1:
        return mine
    parts = [None] * world
    dist.all_gather_object(parts, mine, group=group)
    parts = [p for p in parts if p is not None]
    return tuple(np.concatenate([p[k] for p in parts]) for k in range(4))


def max_over_ranks(value: float, group=None) -> float:
    """Largest `value` over all ranks (timings are reported as the slowest rank's)."""
    import torch
    import torch.distributed as dist
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
