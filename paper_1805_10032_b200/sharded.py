"""The Zeno step for a least-squares parameter vector sharded over several GPUs by column slice.

One process per GPU (torch.distributed).  Rank g owns the columns [lo_g, hi_g) of x, of every candidate row
of V and of the batch matrix A.  Definition 2's score needs A (x - gamma v_i) - y, which is a sum over the
slices, so the ranks exchange one small array -- (m + 1) (n_r + 1) doubles: the slices' products A_s x_s,
A_s v_i and their shares of ||v_i||^2 -- with a single all-reduce.  After that every rank holds the same
scores, ranks them the same way (Definition 3) and averages its own columns of the selected rows; the
aggregate stays sharded like x and nothing else crosses the links.

This module only moves arguments: the products, the finish, the ranking and the mean run in the CUDA library
(zeno_score_partial, zeno_score_from_sums, zeno_select, zeno_aggregate); the all-reduce is the process
group's (NCCL between GPUs).
"""
from __future__ import annotations

from typing import List, Tuple


def column_slices(d: int, world: int, align: int = 32) -> List[Tuple[int, int]]:
    """Contiguous column ranges [lo, hi) for `world` ranks that cover [0, d): equal up to `align` columns
    (slice starts stay on 128-byte boundaries for binary32 rows), the last rank takes the remainder, and a
    rank may be left empty when d is small."""
    if d < 0 or world < 1 or align < 1:
        raise ValueError("bad slicing arguments")
    per = -(-d // world)                     # ceil
    per = -(-per // align) * align           # rounded up to the alignment
    out = []
    for g in range(world):
        lo = min(d, g * per)
        hi = min(d, lo + per)
        out.append((lo, hi))
    return out


def sharded_step(handle, x_s, V_s, A_s, y, gamma, rho, b, group=None, dist=None):
    """One Zeno step on this rank's slice.

    handle: a least-squares handle made for the slice length (handle.d == x_s.numel());
    x_s [d_s], V_s [m, ldv_s], A_s [n_r, d_s] contiguous, y [n_r]: this rank's device tensors.
    Returns (out_s [d_s] float32, scores [m], idx [m - b]); scores and idx are identical on every rank.
    """
    sums = handle.score_partial(x_s, V_s, A_s)
    if dist is None:
        import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
    scores, _, _ = handle.score_from_sums(sums, y, gamma, rho)
    idx = handle.select(scores, b)
    out_s = handle.aggregate(V_s, idx)
    return out_s, scores, idx
