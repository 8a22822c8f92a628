"""Column sharding across GPUs (host logic only).

The mixing matrix acts on rows (nodes) and the gradient and noise are element-wise,
keyed by the global column index, so disjoint column ranges evolve independently:
each rank owns a range, sets its column offset, and no data-path collective is needed.
Only scalar diagnostics (consensus distance, loss) are summed over ranks.
"""
from __future__ import annotations


def weak_shard_offset(rank: int, d: int) -> int:
    """Weak scaling: every rank holds d columns of a (world * d)-column problem.
    Offsets are multiples of 4 (one generator call covers 4 columns)."""
    return rank * ((d + 3) // 4 * 4)


def split_columns(d_total: int, world: int):
    """Strong scaling: cut [0, d_total) into `world` contiguous ranges whose starts are
    multiples of 4; returns [(col0, width), ...] (widths may be 0 for tiny d_total)."""
    groups = (d_total + 3) // 4
    base, extra = divmod(groups, world)
    out, g0 = [], 0
    for r in range(world):
        g = base + (1 if r < extra else 0)
        c0 = min(g0 * 4, d_total)
        c1 = min((g0 + g) * 4, d_total)
        out.append((c0, c1 - c0))
        g0 += g
    return out


def all_reduce_sum(value: float, group=None) -> float:
    """Sum a host scalar over ranks (consensus distance and loss are sums over columns)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64)
    if dist.get_backend(group) == "nccl":
        t = t.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t.item())
