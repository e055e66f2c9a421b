"""CPU-only tests of the library's host side through the C ABI: exported symbols, mesh, layout
legality, slice index maps (bit-exact against the oracle's independent implementation), einsum
planning (reduce groups, distinct slices, kernel family) and cost counts (against the oracle and
the paper's closed forms).  No kernel is launched."""
import ctypes
import itertools
import json
import os
import re

import numpy as np
import pytest

import paper_1811_02084_b200 as mtf
from oracle import IllegalLayout, Layout, Mesh, NotDivisible, OracleError, cost
import seeded_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_statements.json")))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mtf.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = sorted(set(re.findall(r"\b(mtf_[a-z0-9_]+)\s*\((?!\*)", header)))      # (function declarations, not function-pointer typedefs)
    assert len(names) >= 25
    lib = ctypes.CDLL(mtf.binding.LIB_PATH)
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing


def test_status_strings():
    assert mtf.mtf_status_string(0) == "MTF_OK"
    assert mtf.mtf_status_string(5) == "MTF_ERR_ILLEGAL_LAYOUT"
    assert mtf.mtf_status_string(10) == "MTF_ERR_TIMEOUT"


def test_mesh_coords_match_oracle():
    for shape in ([4], [2, 3], [2, 2, 2], [4, 8], [2, 3, 2, 2]):
        dims = [(f"m{i}", s) for i, s in enumerate(shape)]
        m, o = mtf.mtf_mesh_create(dims), Mesh(dims)
        assert mtf.mtf_mesh_size(m) == o.P
        for p in range(o.P):
            assert tuple(mtf.mtf_mesh_coords(m, p)) == o.coords(p)
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_mesh_create([("a", 2), ("a", 2)])
    assert e.value.code == "MTF_ERR_DUPLICATE_DIM"
    with pytest.raises(mtf.MtfError):
        mtf.mtf_mesh_create([("a", 0)])
    with pytest.raises(mtf.MtfError):
        mtf.mtf_mesh_coords(mtf.mtf_mesh_create([("a", 2)]), 2)


def test_empty_dimensions_are_refused():
    L = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 2)]), [("batch", "all")])
    a, b = mtf.desc([("batch", 4), ("k", 0)], "bf16"), mtf.desc([("k", 0), ("j", 8)], "bf16")
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_plan(L, [a, b], mtf.desc([("batch", 4), ("j", 8)], "bf16"))
    assert e.value.code == "MTF_ERR_INVALID_ARG"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_layout_check_tensor(L, [("batch", 0)])
    assert e.value.code == "MTF_ERR_INVALID_ARG"


def both(mesh_dims, rules):
    return mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules), Layout(Mesh(mesh_dims), rules)


def test_slice_maps_bit_exact_exhaustive_small():
    tensor = [("batch", 4), ("hidden", 6), ("io", 12)]
    for mesh_dims in ([("a", 2)], [("a", 2), ("b", 3)], [("a", 2), ("b", 2), ("c", 3)]):
        mnames = [n for n, _ in mesh_dims]
        for assign in itertools.product([None] + mnames, repeat=3):
            rules = [(t, m) for (t, _), m in zip(tensor, assign) if m is not None]
            L, O = both(mesh_dims, rules)
            for p in range(O.mesh.P):
                try:
                    want = O.slice_box(tensor, p)
                except OracleError as ex:
                    with pytest.raises(mtf.MtfError) as e:
                        mtf.mtf_slice_map(L, tensor, p)
                    assert e.value.code == ex.code
                    continue
                offs, sizes = mtf.mtf_slice_map(L, tensor, p)
                assert (offs, sizes) == (list(want[0]), list(want[1]))


def test_slice_maps_bit_exact_seeded_random():
    rng = np.random.default_rng(123)          # only picks shapes; no tensor data involved
    names = ["batch", "length", "heads", "d_k", "d_model", "d_ff", "vocab"]
    for trial in range(200):
        nm = int(rng.integers(1, 5))
        mesh_dims = [(f"m{j}", int(rng.choice([1, 2, 3, 4, 8]))) for j in range(nm)]
        nt = int(rng.integers(1, 6))
        tnames = list(rng.choice(names, size=nt, replace=False))
        rules = [(t, f"m{int(rng.integers(0, nm))}") for t in tnames if rng.random() < 0.6]
        dims = [(t, int(rng.choice([1, 2, 3, 4, 6, 8, 12, 16, 24, 48, 96]))) for t in tnames]
        L, O = both(mesh_dims, rules)
        for p in range(O.mesh.P):
            try:
                want = O.slice_box(dims, p)
            except OracleError as ex:
                with pytest.raises(mtf.MtfError) as e:
                    mtf.mtf_slice_map(L, dims, p)
                assert e.value.code == ex.code, (mesh_dims, rules, dims)
                break
            offs, sizes = mtf.mtf_slice_map(L, dims, p)
            assert (offs, sizes) == (list(want[0]), list(want[1])), (mesh_dims, rules, dims, p)


def test_paper_legal_and_illegal_layouts():
    mesh = mtf.mtf_mesh_create([("all", 4)])
    h = [("batch", 8), ("hidden", 16)]
    mtf.mtf_layout_check_tensor(mtf.mtf_layout(mesh, []), h)                          # Section 8.4
    bad = mtf.mtf_layout(mesh, [("batch", "all"), ("hidden", "all")])                # Section 8.5
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_layout_check_tensor(bad, h)
    assert e.value.code == "MTF_ERR_ILLEGAL_LAYOUT"
    mtf.mtf_layout_check_tensor(bad, [("batch", 8), ("io", 4)])
    tr = mtf.mtf_layout(mesh, [("vocab", "all"), ("d_ff", "all"), ("heads", "all")])   # Section 9
    for d in ([("batch", 2), ("length", 3), ("d_ff", 8)], [("d_model", 4), ("heads", 4), ("d_k", 2)], [("vocab", 8), ("d_model", 4)]):
        mtf.mtf_layout_check_tensor(tr, d)
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_layout_check_tensor(mtf.mtf_layout(mesh, [("batch", "all")]), [("batch", 6)])
    assert e.value.code == "MTF_ERR_NOT_DIVISIBLE"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_layout(mesh, [("batch", "nope")])
    assert e.value.code == "MTF_ERR_UNKNOWN_DIM"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_layout(mesh, [("batch", "all"), ("batch", "all")])
    assert e.value.code == "MTF_ERR_INVALID_ARG"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_layout_check_tensor(tr, [("batch", 2), ("batch", 3)])
    assert e.value.code == "MTF_ERR_DUPLICATE_DIM"


def test_einsum_plan_errors():
    L, _ = both([("all", 2)], [("i", "all"), ("j", "all")])
    a, b = mtf.desc([("i", 4), ("k", 4)], "f32"), mtf.desc([("k", 4), ("j", 4)], "f32")
    with pytest.raises(mtf.MtfError) as e:                      # iteration space not injective
        mtf.mtf_einsum_plan(L, [a, b], mtf.desc([("k", 4)], "f32"))
    assert e.value.code == "MTF_ERR_ILLEGAL_LAYOUT"
    L2, _ = both([("all", 2)], [])
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_plan(L2, [a, b], mtf.desc([("i", 4), ("z", 4)], "f32"))
    assert e.value.code == "MTF_ERR_UNKNOWN_DIM"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_plan(L2, [a, mtf.desc([("k", 5), ("j", 4)], "f32")], mtf.desc([("i", 4), ("j", 4)], "f32"))
    assert e.value.code == "MTF_ERR_SIZE_MISMATCH"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_plan(L2, [a, b, a], mtf.desc([("i", 4), ("j", 4)], "f32"))
    assert e.value.code == "MTF_ERR_UNSUPPORTED"
    with pytest.raises(mtf.MtfError) as e:                      # bias over a dim the output lacks
        mtf.mtf_einsum_plan(L2, [a, b], mtf.desc([("i", 4), ("j", 4)], "f32"), mtf.Epilogue(bias=mtf.desc([("k", 4)], "f32")))
    assert e.value.code == "MTF_ERR_UNKNOWN_DIM"


def example_descs(sym, dtype="f32"):
    b, d_io, d_h = sym["b"], sym["d_io"], sym["d_h"]
    d = {"x": [("batch", b), ("io", d_io)], "w": [("io", d_io), ("hidden", d_h)], "v": [("hidden", d_h), ("io", d_io)],
         "h": [("batch", b), ("hidden", d_h)], "y": [("batch", b), ("io", d_io)]}
    eins = {"h": (["x", "w"], "h"), "y": (["h", "v"], "y"), "dh": (["y", "v"], "h"), "dv": (["h", "y"], "v"),
            "dw": (["x", "h"], "w"), "dx": (["h", "w"], "y")}
    return d, eins


SYM = dict(b=48, d_io=12, d_h=36, n=4, r=2, c=3, p=2)


def ev(expr):
    return int(eval(str(expr), {}, dict(SYM)))


@pytest.mark.parametrize("row", GOLD["table1"]["rows"], ids=lambda r: str(r["layout"]))
def test_plan_cost_equals_oracle_and_table1(row):
    mesh_dims = [(n, ev(s)) for n, s in row["mesh"]]
    rules = [tuple(r) for r in row["layout"]]
    L, O = both(mesh_dims, rules)
    d, eins = example_descs(SYM)
    msgs = set()
    for name, (ins, out) in eins.items():
        plan = mtf.mtf_einsum_plan(L, [mtf.desc(d[i], "f32") for i in ins], mtf.desc(d[out], "f32"))
        got = mtf.mtf_plan_cost(plan)
        want = cost.einsum_cost(O, [d[i] for i in ins], [n for n, _ in d[out]])
        assert got["macs_per_proc"] == want["macs_per_proc"]
        assert got["allreduce_values"] == want["allreduce_values"]
        assert got["slice_elems"] == want["slice_elems"]
        assert got["n_reduce_mesh_dims"] == len(want["reduce_mesh_dims"])
        info = mtf.mtf_plan_info(plan)
        assert info["reduce_mesh_dim_mask"] == sum(1 << j for j in want["reduce_mesh_dims"])
        assert info["n_slices"] * want["replication"] == O.mesh.P
        if got["allreduce_values"]:
            msgs.add((info["reduce_mesh_dim_mask"], got["allreduce_values"]))
        if name == "h":
            assert got["macs_per_proc"] == ev(row["comp"])
            assert got["slice_elems"] == ev(row["memory"])
    assert sum(v for _, v in msgs) == ev(row["comm"])


def test_allreduce_value_counts_of_section_8():
    d, eins = example_descs(SYM)
    for case in GOLD["allreduce_values_per_processor"]:
        L, _ = both([(n, ev(s)) for n, s in case["mesh"]], [tuple(r) for r in case["layout"]])
        total = 0
        for ins, out in eins.values():
            plan = mtf.mtf_einsum_plan(L, [mtf.desc(d[i], "f32") for i in ins], mtf.desc(d[out], "f32"))
            total += mtf.mtf_plan_cost(plan)["allreduce_values"]
        assert total == ev(case["matrices_only"])


def test_appendix_b_ratios_from_the_plan():
    g = GOLD["appendix_b"]
    u = g["u"]
    a, b, c = mtf.desc([("i", u), ("k", u)], "f32"), mtf.desc([("k", u), ("j", u)], "f32"), mtf.desc([("i", u), ("j", u)], "f32")
    for key in ("two_d", "three_d"):
        L, _ = both([tuple(m) for m in g[key]["mesh"]], [tuple(r) for r in g[key]["layout"]])
        got = mtf.mtf_plan_cost(mtf.mtf_einsum_plan(L, [a, b], c))
        assert got["slice_elems"] == int(eval(g[key]["footprint"], {}, {"u": u}))
        num, den = int(eval(g[key]["ratio_num"], {}, {"u": u})), int(g[key]["ratio_den"])
        assert 2 * got["macs_per_proc"] * den == got["slice_elems"] * num


def test_kernel_family_and_reduce_groups_of_the_benchmark_shapes():
    bf = "bf16"
    x = mtf.desc([("batch", 32), ("length", 256), ("d_model", 1024)], bf)
    w = mtf.desc([("d_model", 1024), ("d_ff", 4096)], bf)
    v = mtf.desc([("d_ff", 4096), ("d_model", 1024)], bf)
    h = mtf.desc([("batch", 32), ("length", 256), ("d_ff", 4096)], bf)
    dw = mtf.desc([("d_model", 1024), ("d_ff", 4096)], "f32")
    mesh8 = [("all", 8)]
    for rules, y_group, dw_group in (([], 1, 1), ([("batch", "all")], 1, 8), ([("d_ff", "all")], 8, 1)):
        L, _ = both(mesh8, rules)
        for ins, out, group in (([x, w], h, 1), ([h, v], x, y_group), ([x, h], dw, dw_group)):
            info = mtf.mtf_plan_info(mtf.mtf_einsum_plan(L, ins, out))
            assert info["kernel_kind"] == mtf.MTF_KERNEL_TCGEN05
            assert info["group_size"] == group
            assert info["n_slices"] == (8 if rules else 1)
            assert info["reduce_mode"] == (mtf.MTF_REDUCE_NONE if group == 1 else mtf.MTF_REDUCE_CHAINED)
    # attention on mesh [4,4]: batch -> rows, heads -> cols
    L, _ = both([("rows", 4), ("cols", 4)], [("batch", "rows"), ("heads", "cols")])
    q = mtf.desc([("batch", 16), ("length", 512), ("heads", 16), ("d_k", 64)], bf)
    k = mtf.desc([("batch", 16), ("memory_length", 512), ("heads", 16), ("d_k", 64)], bf)
    lg = mtf.desc([("batch", 16), ("heads", 16), ("length", 512), ("memory_length", 512)], bf)
    info = mtf.mtf_plan_info(mtf.mtf_einsum_plan(L, [q, k], lg))
    assert info == {"kernel_kind": 1, "reduce_mode": 0, "n_slices": 16, "group_size": 1, "reduce_mesh_dim_mask": 0}
    wo = mtf.desc([("heads", 16), ("d_v", 64), ("d_model", 1024)], bf)
    o = mtf.desc([("batch", 16), ("length", 512), ("heads", 16), ("d_v", 64)], bf)
    y = mtf.desc([("batch", 16), ("length", 512), ("d_model", 1024)], bf)
    info = mtf.mtf_plan_info(mtf.mtf_einsum_plan(L, [o, wo], y))
    assert info["group_size"] == 4 and info["reduce_mesh_dim_mask"] == 2 and info["kernel_kind"] == 1
    # fp32 toy: generic kernel
    L, _ = both([("rows", 2), ("cols", 2)], [("batch", "rows"), ("hidden", "cols")])
    info = mtf.mtf_plan_info(mtf.mtf_einsum_plan(L, [mtf.desc([("batch", 8), ("io", 64)], "f32"), mtf.desc([("io", 64), ("hidden", 256)], "f32")],
                                                 mtf.desc([("batch", 8), ("hidden", 256)], "f32")))
    assert info["kernel_kind"] == mtf.MTF_KERNEL_SIMT and info["n_slices"] == 4


def test_forced_choices_are_validated():
    L, _ = both([("all", 2)], [("k", "all")])
    a, b, c = mtf.desc([("i", 128), ("k", 256)], "f32"), mtf.desc([("k", 256), ("j", 128)], "f32"), mtf.desc([("i", 128), ("j", 128)], "f32")
    mtf.mtf_plan_force(1, -1)
    try:
        with pytest.raises(mtf.MtfError) as e:
            mtf.mtf_einsum_plan(L, [a, b], c)                       # fp32 operands cannot take the bf16 tensor-core path
        assert e.value.code == "MTF_ERR_UNSUPPORTED"
    finally:
        mtf.mtf_plan_force(-1, -1)
    with pytest.raises(mtf.MtfError):
        mtf.mtf_plan_force(7, 0)


def test_exec_rejects_null_data_and_wrong_shapes_before_any_launch():
    L, _ = both([("all", 1)], [])
    a, b, c = mtf.desc([("i", 4), ("k", 4)], "f32"), mtf.desc([("k", 4), ("j", 4)], "f32"), mtf.desc([("i", 4), ("j", 4)], "f32")
    plan = mtf.mtf_einsum_plan(L, [a, b], c)
    n0 = mtf.mtf_launch_count()
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_exec(plan, [a, b], c)                        # descriptors carry no data
    assert e.value.code == "MTF_ERR_INVALID_ARG"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_exec(plan, [a, mtf.desc([("k", 4), ("j", 5)], "f32")], c)
    assert e.value.code == "MTF_ERR_SIZE_MISMATCH"
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum(L, "i k, k j -> j i", [a, b], c)
    assert e.value.code == "MTF_ERR_INVALID_ARG"
    assert mtf.mtf_launch_count() == n0
