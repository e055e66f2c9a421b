"""TEST INFRASTRUCTURE.  Per-processor cost counts of one lowered einsum.

Table 1 and Sections 8.1-8.3 count, per processor, the multiply-adds of the local einsum and the
number of values that enter an Allreduce (one output slice whenever a split dimension is reduced
out).  Appendix B counts the elements a processor must access: the sizes of the projections of its
part of the iteration space onto each operand, i.e. the sizes of its input and output slices.
"""
from __future__ import annotations

from .named import resolve_out_dims, union_dims


def _prod(xs):
    r = 1
    for x in xs:
        r *= int(x)
    return r


def einsum_cost(layout, in_dim_lists, out_names):
    """Returns a dict:
    macs_per_proc          product of the local extents of the whole iteration space
    allreduce_values       elements of the local output slice if a reduced-out dim is split, else 0
    reduce_mesh_dims       sorted mesh-dim indices the Allreduce runs over
    slice_elems            local elements of inputs plus output (Appendix B footprint)
    used_mesh_dims         mesh dims some dimension of the iteration space is split over
    replication            processors doing identical work = P / prod(sizes of used mesh dims)
    """
    out_dims = resolve_out_dims(in_dim_lists, out_names)
    space = union_dims(list(in_dim_lists) + [out_dims])
    layout.check_iteration_space(list(in_dim_lists) + [out_dims])
    macs = _prod(t for _, t in layout.slice_dims(tuple(space)))
    out_names_l = [n for n, _ in out_dims]
    over = sorted({layout.mesh_dim_of(n) for n, _ in space
                   if n not in out_names_l and layout.mesh_dim_of(n) is not None})
    out_slice = _prod(t for _, t in layout.slice_dims(out_dims))
    foot = out_slice + sum(_prod(t for _, t in layout.slice_dims(tuple(d))) for d in in_dim_lists)
    used = sorted({layout.mesh_dim_of(n) for n, _ in space if layout.mesh_dim_of(n) is not None})
    repl = layout.mesh.P // _prod(layout.mesh.shape[j] for j in used)
    return {"macs_per_proc": macs, "allreduce_values": out_slice if over else 0,
            "reduce_mesh_dims": over, "slice_elems": foot, "used_mesh_dims": used, "replication": repl}
