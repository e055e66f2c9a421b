"""Pins for the oracle's mesh, layout legality, slice boxes, lowering and cost counts (CPU only).

Pinned against what the paper states (tests/golden/paper_statements.json: slice shapes, where an
Allreduce happens, values allreduced, Table 1, Appendix B) and against invariants: the slices of a
tensor partition it, and every legal layout gives exactly the un-split result (Section 8: "each
will produce identical results") - checked with small-integer inputs so fp64 sums are exact in any
order.
"""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import (NT, DenseOps, IllegalLayout, Layout, LoweredOps, Mesh, NotDivisible, OracleError,
                    UnknownDim, blocks, cost)
import seeded_inputs as si

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_statements.json")))
SYM = dict(b=48, d_io=12, d_h=36, n=4, r=2, c=3, p=2)


def ev(expr, sym=SYM):
    return int(eval(str(expr), {}, dict(sym)))


def build(mesh, layout, sym=SYM):
    m = Mesh([(n, ev(s, sym)) for n, s in mesh])
    return m, Layout(m, [tuple(r) for r in layout])


def example_dims(sym=SYM):
    b, d_io, d_h = sym["b"], sym["d_io"], sym["d_h"]
    return {"x": [("batch", b), ("io", d_io)], "w": [("io", d_io), ("hidden", d_h)], "bias": [("hidden", d_h)],
            "v": [("hidden", d_h), ("io", d_io)], "h": [("batch", b), ("hidden", d_h)], "y": [("batch", b), ("io", d_io)]}


# ---- mesh ---------------------------------------------------------------------------------------

def test_processor_rank_is_row_major_last_dim_fastest():
    m = Mesh([("rows", 2), ("cols", 3)])
    assert [m.coords(p) for p in range(6)] == [(0, 0), (0, 1), (0, 2), (1, 0), (1, 1), (1, 2)]
    assert all(m.rank(m.coords(p)) == p for p in range(6))
    # groups of a partitioned Allreduce: over cols = the processors of one row
    assert m.group(4, {1}) == [3, 4, 5]
    assert m.group(4, {0}) == [1, 4]
    assert m.group(4, {0, 1}) == list(range(6))
    assert m.group(4, set()) == [4]


def test_same_processors_viewed_as_different_meshes():
    # Section 2: 512 processors as [16,16,2], [32,16] or [512]
    for shape in ([16, 16, 2], [32, 16], [512]):
        assert Mesh([(f"m{i}", s) for i, s in enumerate(shape)]).P == 512


# ---- slice shapes printed in the paper ------------------------------------------------------------

@pytest.mark.parametrize("case", GOLD["slice_shapes"], ids=lambda c: c["cite"][:20])
def test_slice_shapes_from_paper(case):
    mesh, lay = build(case["mesh"], case["layout"])
    dims = example_dims()
    for name, shape in case["tensors"].items():
        for p in range(mesh.P):
            _, sizes = lay.slice_box(dims[name], p)
            assert sizes == [ev(s) for s in shape], (name, p)


def test_2d_layout_rows_share_x_and_columns_share_w():
    mesh, lay = build([["rows", "r"], ["cols", "c"]], [["batch", "rows"], ["hidden", "cols"]])
    dims = example_dims()
    for p in range(mesh.P):
        for q in range(mesh.P):
            same_row = mesh.coords(p)[0] == mesh.coords(q)[0]
            same_col = mesh.coords(p)[1] == mesh.coords(q)[1]
            assert (lay.slice_box(dims["x"], p) == lay.slice_box(dims["x"], q)) == same_row
            assert (lay.slice_box(dims["w"], p) == lay.slice_box(dims["w"], q)) == same_col


def test_slices_partition_the_tensor_and_index_payload():
    mesh = Mesh([("rows", 2), ("cols", 3), ("planes", 2)])
    lay = Layout(mesh, [("batch", "rows"), ("hidden", "cols"), ("io", "planes")])
    dims = [("batch", 4), ("hidden", 6), ("io", 2)]
    total = 4 * 6 * 2
    payload = np.arange(total, dtype=np.float64).reshape(4, 6, 2)
    seen = np.zeros(total, dtype=np.int64)
    for p in range(mesh.P):
        idx = lay.global_flat_indices(dims, p)
        sl = lay.slice_of(dims, payload, p)
        assert np.array_equal(sl.reshape(-1), idx.astype(np.float64))   # payload = own flat index
        seen[idx] += 1
    assert (seen == 1).all()            # all three dims split over all three mesh dims: no replication
    # contiguous block stripes: processor with coordinate c gets [c*s/m, (c+1)*s/m)
    offs, sizes = lay.slice_box(dims, mesh.rank((1, 2, 0)))
    assert offs == [2, 4, 0] and sizes == [2, 2, 1]
    # replicated tensor: every processor holds everything
    lay2 = Layout(mesh, [("batch", "rows")])
    for p in range(mesh.P):
        assert lay2.slice_box([("hidden", 6)], p) == ([0], [6])


# ---- legality --------------------------------------------------------------------------------------

def test_legal_and_illegal_layouts_of_the_paper():
    mesh = Mesh([("all", 4)])
    dims = example_dims()
    Layout(mesh, []).tensor_layout(dims["h"])                                    # empty layout is legal
    bad = Layout(mesh, [("batch", "all"), ("hidden", "all")])                       # Section 8.5
    with pytest.raises(IllegalLayout):
        bad.tensor_layout(dims["h"])
    bad.tensor_layout(dims["x"])         # x has only one of the two dims: its own layout is fine
    # Section 9: vocab, d_ff, heads all on one mesh dim is legal because no tensor has two of them
    tr = Layout(mesh, [("vocab", "all"), ("d_ff", "all"), ("heads", "all")])
    for d in ([("batch", 2), ("length", 3), ("d_ff", 8)], [("d_model", 4), ("heads", 4), ("d_k", 2)],
              [("vocab", 8), ("d_model", 4)], [("d_model", 4), ("d_ff", 8)]):
        tr.tensor_layout(d)
    with pytest.raises(NotDivisible):
        Layout(mesh, [("batch", "all")]).tensor_layout([("batch", 6)])
    with pytest.raises(UnknownDim):
        Layout(mesh, [("batch", "nope")])
    with pytest.raises(OracleError):
        Layout(mesh, [("batch", "all"), ("batch", "all")])


def test_einsum_iteration_space_must_be_injective():
    # A[i,k] . B[k,j] with i and j on the same mesh dim: no single tensor is illegal but each
    # processor would only hold matching blocks of i and j -> rejected for the operation.
    mesh = Mesh([("all", 2)])
    lay = Layout(mesh, [("i", "all"), ("j", "all")])
    ops = LoweredOps(lay)
    a = ops.lower(NT([("i", 2), ("k", 2)], np.ones((2, 2))))
    b = ops.lower(NT([("k", 2), ("j", 2)], np.ones((2, 2))))
    with pytest.raises(IllegalLayout):
        ops.einsum([a, b], ["k"])


# ---- the invariant: every legal layout gives exactly the un-split result ---------------------------

def all_layouts(tensor_dims, mesh):
    """Every partial injective map from tensor-dim names to mesh-dim names."""
    names = list(tensor_dims)
    for assign in itertools.product([None] + list(mesh.names), repeat=len(names)):
        rules = [(n, m) for n, m in zip(names, assign) if m is not None]
        yield rules


@pytest.mark.parametrize("mesh_dims", [[("a", 2)], [("a", 2), ("b", 2)], [("a", 2), ("b", 3)], [("a", 2), ("b", 2), ("c", 2)]])
def test_every_layout_gives_identical_result_matmul(mesh_dims):
    mesh = Mesh(mesh_dims)
    sizes = {"i": 12, "j": 6, "k": 12}
    A = NT([("i", 12), ("k", 12)], si.small_integers(11, "A", (12, 12)))
    B = NT([("k", 12), ("j", 6)], si.small_integers(11, "B", (12, 6)))
    want = DenseOps().einsum([A, B], ["i", "j"]).a
    n_legal = n_illegal = 0
    for rules in all_layouts(sizes, mesh):
        lay = Layout(mesh, rules)
        ops = LoweredOps(lay)
        try:
            got = ops.to_global(ops.einsum([ops.lower(A), ops.lower(B)], ["i", "j"]))
        except IllegalLayout:
            n_illegal += 1
            assert len({m for _, m in rules}) < len(rules)     # only when two dims share a mesh dim
            continue
        n_legal += 1
        assert np.array_equal(got.a, want), rules
        # an Allreduce happened exactly when k is split
        assert (len(ops.allreduce_log) == 1) == any(t == "k" for t, _ in rules)
    assert n_legal > 0
    if len(mesh_dims) == 1:
        assert n_legal == 4 and n_illegal == 4


def test_every_layout_gives_identical_result_batched_and_multi_dim():
    # q[b,l,h,k] = sum_d x[b,l,d] wq[d,h,k]  and  lg[b,h,l,m] = sum_k q kk
    mesh = Mesh([("a", 2), ("b", 2)])
    x = NT([("batch", 2), ("length", 4), ("d_model", 4)], si.small_integers(12, "x", (2, 4, 4)))
    wq = NT([("d_model", 4), ("heads", 2), ("d_k", 2)], si.small_integers(12, "wq", (4, 2, 2)))
    kk = NT([("batch", 2), ("memory_length", 4), ("heads", 2), ("d_k", 2)], si.small_integers(12, "kk", (2, 4, 2, 2)))
    d = DenseOps()
    q_want = d.einsum([x, wq], ["batch", "length", "heads", "d_k"])
    lg_want = d.einsum([q_want, kk], ["batch", "heads", "length", "memory_length"])
    names = ["batch", "length", "d_model", "heads", "d_k", "memory_length"]
    count = 0
    for rules in all_layouts(names, mesh):
        lay = Layout(mesh, rules)
        ops = LoweredOps(lay)
        try:
            q = ops.einsum([ops.lower(x), ops.lower(wq)], ["batch", "length", "heads", "d_k"])
            lg = ops.einsum([q, ops.lower(kk)], ["batch", "heads", "length", "memory_length"])
        except IllegalLayout:
            continue
        count += 1
        assert np.array_equal(ops.to_global(q).a, q_want.a)
        assert np.array_equal(ops.to_global(lg).a, lg_want.a)
    assert count >= 30


def test_lowered_reductions_and_broadcast():
    mesh = Mesh([("a", 2), ("b", 2)])
    x = NT([("batch", 4), ("hidden", 6)], si.small_integers(13, "x", (4, 6)))
    bias = NT([("hidden", 6)], si.small_integers(13, "bias", (6,)))
    d = DenseOps()
    for rules in all_layouts(["batch", "hidden"], mesh):
        if len({m for _, m in rules}) < len(rules):
            continue
        ops = LoweredOps(Layout(mesh, rules))
        lx, lb = ops.lower(x), ops.lower(bias)
        assert np.array_equal(ops.to_global(ops.add(lx, lb)).a, d.add(x, bias).a)
        assert np.array_equal(ops.to_global(ops.reduce_sum(lx, ["hidden"])).a, x.a.sum(0))
        assert np.array_equal(ops.to_global(ops.reduce_max(lx, ["batch"])).a, x.a.max(1))
        assert np.array_equal(ops.to_global(ops.reduce_sum(lx, [])).a, x.a.sum())


# ---- where the Allreduce happens, and how many values -----------------------------------------------

def run_example(mesh, lay, sym, with_bias=True):
    dims = example_dims(sym)
    t = {k: NT(v, si.small_integers(14, k, [s for _, s in v], -2, 2)) for k, v in dims.items() if k in ("x", "w", "bias", "v")}
    dy = NT(dims["y"], si.small_integers(14, "dy", [s for _, s in dims["y"]], -2, 2))
    ops = LoweredOps(lay)
    L = {k: ops.lower(v) for k, v in t.items()}
    f = blocks.ffn_forward(ops, L["x"], L["w"], L["bias"] if with_bias else None, L["v"])
    n_fwd = len(ops.allreduce_log)
    g = blocks.ffn_backward(ops, L["x"], L["w"], L["v"], f["h"], ops.lower(dy))
    # dense reference
    dn = DenseOps()
    fd = blocks.ffn_forward(dn, t["x"], t["w"], t["bias"] if with_bias else None, t["v"])
    gd = blocks.ffn_backward(dn, t["x"], t["w"], t["v"], fd["h"], dy)
    for k in ("y", "h"):
        assert np.array_equal(ops.to_global(f[k]).a, fd[k].a), k
    for k in ("dx", "dw", "dv", "dbias"):
        assert np.array_equal(ops.to_global(g[k]).a, gd[k].a), k
    return ops.allreduce_log[:n_fwd], ops.allreduce_log[n_fwd:]


@pytest.mark.parametrize("case", GOLD["where_allreduce_happens"], ids=lambda c: c["cite"][:14])
def test_where_allreduce_happens(case):
    sym = dict(b=8, d_io=4, d_h=8)
    mesh, lay = build(case["mesh"], case["layout"], sym)
    fwd, bwd = run_example(mesh, lay, sym)
    assert len(fwd) == len(case["forward"])
    assert len(bwd) == len(case["backward"])
    if case["layout"] == [["batch", "rows"], ["hidden", "cols"]]:
        assert fwd[0][1] == (1,)                              # y summed over the cols mesh dim
        over = sorted(e[1] for e in bwd)
        assert over == [(0,), (0,), (0,), (1,)]               # dv, dw, dbias over rows; dx over cols


@pytest.mark.parametrize("case", GOLD["allreduce_values_per_processor"], ids=lambda c: c["cite"][:14])
def test_values_allreduced_per_processor(case):
    mesh, lay = build(case["mesh"], case["layout"])
    fwd, bwd = run_example(mesh, lay, SYM)
    total = sum(e[2] for e in fwd + bwd)
    assert total == ev(case["with_bias"])
    mats = sum(e[2] for e in fwd + bwd if e[0] == "einsum")
    assert mats == ev(case["matrices_only"])
    # the same numbers from the cost report, without running anything
    d = example_dims()
    eins = [([d["x"], d["w"]], ["batch", "hidden"]), ([d["h"], d["v"]], ["batch", "io"]),
            ([d["y"], d["v"]], ["batch", "hidden"]), ([d["h"], d["y"]], ["hidden", "io"]),
            ([d["x"], d["h"]], ["io", "hidden"]), ([d["h"], d["w"]], ["batch", "io"])]
    assert sum(cost.einsum_cost(lay, i, o)["allreduce_values"] for i, o in eins) == ev(case["matrices_only"])


def test_table1_columns():
    d = example_dims()
    for row in GOLD["table1"]["rows"]:
        mesh, lay = build(row["mesh"], row["layout"])
        first = cost.einsum_cost(lay, [d["x"], d["w"]], ["batch", "hidden"])
        # computation: multiply-adds per processor of one of the two equal-cost einsums
        assert first["macs_per_proc"] == ev(row["comp"])
        # memory per processor: slices of x, h and w (v has as many elements as w; constants dropped)
        assert first["slice_elems"] == ev(row["memory"])
        # communication: one Allreduce per distinct message size (constants dropped): the distinct
        # output-slice sizes that are allreduced somewhere in forward + backward
        eins = [([d["x"], d["w"]], ["batch", "hidden"]), ([d["h"], d["v"]], ["batch", "io"]),
                ([d["y"], d["v"]], ["batch", "hidden"]), ([d["h"], d["y"]], ["hidden", "io"]),
                ([d["x"], d["h"]], ["io", "hidden"]), ([d["h"], d["w"]], ["batch", "io"])]
        msgs = set()
        for i, o in eins:
            c = cost.einsum_cost(lay, i, o)
            if c["allreduce_values"]:
                msgs.add((tuple(c["reduce_mesh_dims"]), c["allreduce_values"]))
        assert sum(v for _, v in msgs) == ev(row["comm"]), row


def test_appendix_b_footprint_and_ratio():
    g = GOLD["appendix_b"]
    u = g["u"]
    dims = [[("i", u), ("k", u)], [("k", u), ("j", u)]]
    for key in ("two_d", "three_d"):
        mesh, lay = build(g[key]["mesh"], g[key]["layout"], {"u": u})
        c = cost.einsum_cost(lay, dims, ["i", "j"])
        assert c["slice_elems"] == ev(g[key]["footprint"], {"u": u})
        assert 2 * c["macs_per_proc"] == 2 * u ** 3 // 64
        # ratio = flops / footprint
        assert 2 * c["macs_per_proc"] * ev(g[key]["ratio_den"], {"u": u}) == c["slice_elems"] * ev(g[key]["ratio_num"], {"u": u})
    # 3-D: exactly one mesh dim allreduced per einsum (Section 8.3)
    mesh, lay = build(g["three_d"]["mesh"], g["three_d"]["layout"], {"u": u})
    assert len(cost.einsum_cost(lay, dims, ["i", "j"])["reduce_mesh_dims"]) == 1


def test_replication_count_of_the_empty_layout():
    mesh = Mesh([("all", 4)])
    d = example_dims()
    c = cost.einsum_cost(Layout(mesh, []), [d["x"], d["w"]], ["batch", "hidden"])
    assert c["replication"] == 4 and c["allreduce_values"] == 0
    c = cost.einsum_cost(Layout(mesh, [("batch", "all")]), [d["x"], d["w"]], ["batch", "hidden"])
    assert c["replication"] == 1
