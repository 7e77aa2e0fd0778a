"""Coordinate sharding of the aggregation path over several GPUs (one process per GPU).

The vote, the median, the means and the trimmed means are independent per coordinate: each rank
aggregates its own contiguous slab of coordinates and nothing is exchanged.  The Krum family needs
one exchange: squared distances are sums over coordinates, so the ranks' partial f x f matrices are
added with a single all-reduce (at most 128 x 128 doubles) before the - replicated - selection.
The exhaustive worst-case search shards over its subsets instead: every rank searches its share and
the ranks' (c_max, argmax) meet in one gather.

``ops`` is the module that supplies the per-rank operations; it defaults to the CUDA binding.  The
functions here contain only the partitioning and the exchange.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def coordinate_slab(d: int, rank: int, world: int, align: int = 4):
    """[begin, end) of the coordinates rank `rank` of `world` owns.  Slab boundaries are multiples of
    `align` (so every slab starts on a 16-byte boundary for fp32), slabs are contiguous, disjoint and
    cover [0, d), and sizes differ by less than 2 * `align`."""
    if world < 1 or not (0 <= rank < world) or d < 0 or align < 1:
        raise ValueError("bad slab request d=%d rank=%d world=%d" % (d, rank, world))
    units = (d + align - 1) // align
    base, extra = divmod(units, world)
    first = rank * base + min(rank, extra)
    last = first + base + (1 if rank < extra else 0)
    return min(first * align, d), min(last * align, d)


def _world(group=None):
    if dist.is_available() and dist.is_initialized():
        return dist.get_world_size(group)
    return 1


def allreduce_sum_(t: torch.Tensor, group=None) -> torch.Tensor:
    """In-place sum over ranks; identity for a single process."""
    if _world(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def _ops(ops):
    if ops is None:
        from . import binding as ops  # the CUDA path; raises if the library is missing
    return ops


def vote_median(replicas_slab: torch.Tensor, ops=None) -> torch.Tensor:
    """Fused vote + median on this rank's slab [r][f][d_local]; no exchange."""
    return _ops(ops).vote_median(replicas_slab)


def multikrum(voted_slab: torch.Tensor, c: int, m: int, ops=None, group=None):
    """Multi-Krum over coordinate slabs.  Returns (out_slab[d_local], selected[m], dist[f][f])."""
    ops = _ops(ops)
    D = ops.pairdist(voted_slab)
    allreduce_sum_(D, group)
    sel = ops.krum_select(D, c, m)
    return ops.mean_rows(voted_slab, sel), sel, D


def bulyan(voted_slab: torch.Tensor, c: int, ops=None, group=None):
    """Bulyan over coordinate slabs.  Returns (out_slab[d_local], selected[f-2c], dist[f][f])."""
    ops = _ops(ops)
    D = ops.pairdist(voted_slab)
    allreduce_sum_(D, group)
    sel = ops.bulyan_select(D, c)
    theta = voted_slab.shape[0] - 2 * c
    return ops.trimmed_mean(voted_slab, sel, theta - 2 * c), sel, D


def vote_multikrum(replicas_slab: torch.Tensor, c: int, m: int, ops=None, group=None):
    """Multi-Krum from the replicas over coordinate slabs: vote and partial distances in one pass over this
    rank's slab [r][f][d_local], one all-reduce of the f x f matrix, replicated selection, mean of the selected
    voted rows of the slab.  Returns (out_slab[d_local], selected[m], dist[f][f], voted_slab[f][d_local])."""
    ops = _ops(ops)
    voted, D = ops.vote_pairdist(replicas_slab)
    allreduce_sum_(D, group)
    sel = ops.krum_select(D, c, m)
    return ops.mean_rows(voted, sel), sel, D, voted


def vote_bulyan(replicas_slab: torch.Tensor, c: int, ops=None, group=None):
    """Bulyan from the replicas over coordinate slabs.  Returns (out_slab, selected[f-2c], dist, voted_slab)."""
    ops = _ops(ops)
    voted, D = ops.vote_pairdist(replicas_slab)
    allreduce_sum_(D, group)
    sel = ops.bulyan_select(D, c)
    theta = voted.shape[0] - 2 * c
    return ops.trimmed_mean(voted, sel, theta - 2 * c), sel, D, voted


def best_of_shares(shares):
    """The result of the whole search from the shares' (c_max, argmax) pairs: the largest c_max, and among
    equals the lexicographically first argmax.  Shares that received nothing (c_max < 0) do not count."""
    best = None
    for c, arg in shares:
        if c < 0:
            continue
        key = (-int(c), tuple(int(u) for u in arg))
        if best is None or key < best[0]:
            best = (key, int(c), [int(u) for u in arg])
    if best is None:
        raise ValueError("no share of the search evaluated a subset")
    return best[1], best[2]


def worst_case(worker_mask, f: int, r: int, q: int, max_subsets: int = 0, ops=None, group=None):
    """Exhaustive c_max^(q) with the subsets dealt to the ranks (bz_worst_case_part), one all-gather of
    (c_max, argmax).  Returns (c_max, argmax[q] list, n_subsets), the same on every rank and the same as the
    single-GPU search."""
    ops = _ops(ops)
    world = _world(group)
    rank = dist.get_rank(group) if world > 1 else 0
    c, arg, n = ops.worst_case_part(worker_mask, f, r, q, rank, world, max_subsets)
    if world == 1:
        return best_of_shares([(c, arg)]) + (n,)
    shares = [None] * world
    dist.all_gather_object(shares, (int(c), [int(u) for u in arg]), group=group)
    return best_of_shares(shares) + (n,)


def worst_case_mols(l: int, r: int, q: int, max_subsets: int = 0, ops=None, group=None):
    """The same for the orbit search of the MOLS placement (bz_worst_case_mols_part).  Returns (c_max, argmax[q]
    list, n_orbits)."""
    ops = _ops(ops)
    world = _world(group)
    rank = dist.get_rank(group) if world > 1 else 0
    c, arg, n = ops.worst_case_mols_part(l, r, q, rank, world, max_subsets)
    if world == 1:
        return best_of_shares([(c, arg)]) + (n,)
    shares = [None] * world
    dist.all_gather_object(shares, (int(c), [int(u) for u in arg]), group=group)
    return best_of_shares(shares) + (n,)
