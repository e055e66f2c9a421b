"""TEST INFRASTRUCTURE.  Picking a computation layout from the cost counts of Table 1.

The paper lists the automated search for a layout as future work (Section 11) and gives the cost
model it would use: per processor, the multiply-adds of the local einsums ("computation") and the
values entering Allreduces ("communication"), Table 1 and Sections 8.1-8.3; Section 8's discussion
says the ratio communication / computation is what makes a layout network bound.  This module is
the plain exhaustive search over that model: every assignment of the candidate tensor dimensions
to mesh dimensions (or to none), legal for every einsum of the workload (Section 5 injectivity per
tensor, divisibility; the iteration-space reading for each einsum), scored by
    cost = sum over einsums of  macs_per_proc + comm_weight * allreduce_values
with ties broken by the smaller memory footprint (sum of slice elements), then by the order of
enumeration (candidate dimensions in the given order, "unsplit" first, mesh dimensions ascending).
"""
from __future__ import annotations

import itertools

from .cost import einsum_cost
from .mesh import Layout, Mesh
from .named import OracleError


def enumerate_layouts(mesh_dims, names):
    """All maps names -> (mesh-dim name or None), in the canonical enumeration order."""
    choices = [None] + [m for m, _ in mesh_dims]
    for combo in itertools.product(choices, repeat=len(names)):
        yield [(n, m) for n, m in zip(names, combo) if m is not None]


def layout_cost(mesh_dims, rules, einsums, comm_weight):
    """(cost, footprint) of one layout over a list of einsums [(input dim lists, output names)], or
    None when the layout is illegal for any of them."""
    lay = Layout(Mesh(mesh_dims), rules)
    cost, foot = 0.0, 0
    for in_dims, out_names in einsums:
        try:
            c = einsum_cost(lay, in_dims, out_names)
            for d in in_dims:
                lay.tensor_layout(d)
        except OracleError:
            return None
        cost += c["macs_per_proc"] + comm_weight * c["allreduce_values"]
        foot += c["slice_elems"]
    return cost, foot


def choose_layout(mesh_dims, names, einsums, comm_weight):
    """Returns (rules, cost, footprint) of the cheapest legal layout."""
    best = None
    for rules in enumerate_layouts(mesh_dims, names):
        r = layout_cost(mesh_dims, rules, einsums, comm_weight)
        if r is None:
            continue
        if best is None or (r[0], r[1]) < (best[1], best[2]):
            best = (rules, r[0], r[1])
    if best is None:
        raise OracleError("no legal layout")
    return best
