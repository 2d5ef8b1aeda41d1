"""Column sharding of the precomputation over several GPUs (host logic only, no device code).

Algorithm 1's loop over feature-column slabs is independent across all K hops, so rank g of G can take one
slab of columns with the graph replicated: no collective on the data path, only the final placement of the
slabs side by side.  The slab rule is the library's own (widths are multiples of 4 floats so that rows stay
128-bit aligned): w = 4 * ceil(F / (4 G)); rank g owns columns [g w, min(F, (g + 1) w)), which may be empty
for the last ranks when F is small.
"""
from __future__ import annotations


def column_shard(feat_dim: int, world: int, rank: int) -> tuple[int, int]:
    """(first column, one past the last column) of `rank`'s slab."""
    if feat_dim < 1 or world < 1 or not 0 <= rank < world:
        raise ValueError("column_shard: bad arguments")
    w = 4 * (-(-feat_dim // (4 * world)))
    lo = min(feat_dim, rank * w)
    return lo, min(feat_dim, lo + w)


def propagate_column_shard(B, rowptr, colidx, op: int, X, K: int, world: int, rank: int, **plan_kw):
    """This rank's share of X_1..X_K: the K hops of its column slab, computed by a plan of the slab's width on a
    strided view of X (no copy).  Returns (first column, list of K [n, width] device tensors), or (lo, []) for an
    empty slab.  `B` is the binding module."""
    lo, hi = column_shard(X.shape[1], world, rank)
    if hi == lo:
        return lo, []
    plan = B.gnnpre_build_plan(rowptr, colidx, op, hi - lo, **plan_kw)
    try:
        outs, _ = B.gnnpre_propagate(plan, X[:, lo:hi], K)
    finally:
        plan.close()
    return lo, outs
