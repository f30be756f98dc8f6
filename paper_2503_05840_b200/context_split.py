"""Host-side logic for splitting ONE context over several GPUs (one process per GPU): which rows a rank
caches, and the exchange of the per-rank results.  Every rank runs slim_decode_partial on its slice,
the ranks all-gather (lse, u) -- H (d + 1) floats per sequence -- and every rank (or only rank 0) calls
slim_combine_project.  The arithmetic is in the library's kernels; this module only slices index
ranges and moves tensors with torch.distributed (nccl on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

TILE = 16          # a slice starts at a multiple of the kernels' context tile


def shard_rows(length: int, world: int, rank: int) -> tuple[int, int]:
    """Rows [start, stop) of a sequence of `length` rows that rank `rank` of `world` caches: contiguous
    slices of whole tiles, as equal as tiles allow; the last non-empty slice takes the ragged tail."""
    tiles = (length + TILE - 1) // TILE
    t0 = (tiles * rank) // world
    t1 = (tiles * (rank + 1)) // world
    return min(t0 * TILE, length), min(t1 * TILE, length)


def shard_batch(lengths, world: int, rank: int):
    """(first_tile[b], slice_length[b]) for every sequence of a batch."""
    first, count = [], []
    for n in lengths:
        a, b = shard_rows(int(n), world, rank)
        first.append(a // TILE)
        count.append(b - a)
    return first, count


def gather_partials(lse, u, dist=None):
    """All-gather of the ranks' (lse [B, H], u [B, H, d]) into ([R, B, H], [R, B, H, d]).  Without a
    process group (one rank) the inputs are returned with a leading axis of one."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return lse.unsqueeze(0), u.unsqueeze(0)
    world = dist.get_world_size()
    lse_all = torch.empty((world,) + tuple(lse.shape), dtype=lse.dtype, device=lse.device)
    u_all = torch.empty((world,) + tuple(u.shape), dtype=u.dtype, device=u.device)
    for dst, src in ((lse_all, lse), (u_all, u)):
        try:
            dist.all_gather_into_tensor(dst, src.contiguous())
        except (RuntimeError, NotImplementedError):            # a backend without the flat form: gather a list
            parts = [torch.empty_like(src) for _ in range(world)]
            dist.all_gather(parts, src.contiguous())
            dst.copy_(torch.stack(parts))
    return lse_all, u_all
