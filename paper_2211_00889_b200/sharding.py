"""Column sharding across ranks (one process per GPU).

The step is independent per parameter column (columns couple only learners and mini-batches), so a
multi-GPU run gives every rank a contiguous column range of ALL K learners and needs no data-path
collective: the only values ranks must agree on are the K finished counts and MATCHA's activation
word, and both are pure functions of (seed, step) that every rank computes for itself.  What ranks
exchange is timing: a barrier around the timed region and the maximum of the per-rank device time.
"""
from typing import Tuple

TILE = 512  # shard boundaries fall on the pipeline kernel's tile width


def column_shard(P_total: int, world: int, rank: int, tile: int = TILE) -> Tuple[int, int]:
    """[c0, c1) of `rank`: whole tiles are dealt out as evenly as possible; the ragged tail (fewer
    than `tile` columns) goes to the last rank."""
    if world < 1 or not (0 <= rank < world) or P_total < 0:
        raise ValueError("bad shard request")
    n_tiles = P_total // tile
    base, extra = divmod(n_tiles, world)
    t0 = rank * base + min(rank, extra)
    t1 = t0 + base + (1 if rank < extra else 0)
    c0, c1 = t0 * tile, t1 * tile
    if rank == world - 1:
        c1 = P_total
    return c0, c1


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of `value` over all ranks (identity without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def counts_agree(n, device=None) -> bool:
    """True when every rank holds the same finished counts `n` (int array [K])."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return True
    t = torch.as_tensor(n, dtype=torch.int64, device=device if device is not None else "cpu").clone()
    lo, hi = t.clone(), t.clone()
    dist.all_reduce(lo, op=dist.ReduceOp.MIN)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX)
    return bool(torch.equal(lo, hi))
