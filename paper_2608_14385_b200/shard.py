"""Department-sharded execution across GPUs: who holds which departments.

A department (its three shared matrices) together with its experts' private matrices is an
independent unit of a DeaMoE layer (paper Section 3.1), and the layer output of Eq. (3) is a sum over
the selected experts.  So a layer spreads over W GPUs by giving each a contiguous range of
departments; every GPU routes all tokens (the router is replicated), computes the partial sum of its
own departments' experts (`Layer.forward_partial`), one all-reduce of the [B, h] fp32 partial sums
completes Eq. (3), and `Layer.finish_partial` adds the residual and rounds to the activation dtype.
This module holds only the partition arithmetic (host side, no layer arithmetic).
"""


def dept_slice(n_dept, rank, world):
    """Departments [begin, end) of `rank` among `world` ranks: contiguous, sizes differing by at most one
    (the first n_dept % world ranks hold one more).  Needs world <= n_dept."""
    if not (0 <= rank < world <= n_dept):
        raise ValueError(f"cannot split {n_dept} departments over {world} ranks (rank {rank})")
    base, extra = divmod(n_dept, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shared_expert_owner(world):
    """The one rank whose slice carries the always-on shared expert: the last, which holds the fewest
    departments when they do not divide evenly."""
    return world - 1


def slice_shape(shape, rank, world):
    """The LayerShape rank `rank` creates its slice with (the shared expert on its owner only; the
    residual flag stays: forward_partial never adds it, finish_partial adds it once) and its
    department range."""
    lo, hi = dept_slice(shape.n_dept, rank, world)
    own = shape.n_shared and rank == shared_expert_owner(world)
    return shape.with_(n_shared=1 if own else 0, shared_ffn=shape.shared_ffn if own else 0), (lo, hi)
