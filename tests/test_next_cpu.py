"""Host logic of the rows beyond the blocks, through the C ABI against the oracle: the reshape
patterns and element counts of Section 6.1 (bit-exact), and the layout search over Table 1's counts
(same layout, same cost, same footprint as the oracle's own exhaustive search)."""
import pytest

import paper_1811_02084_b200 as mtf
import seeded_inputs as si
from oracle import NT, Layout, LoweredOps, Mesh, chooser
from oracle.named import OracleError

PATTERN = {"allgather": mtf.MTF_RESHAPE_ALLGATHER, "slice": mtf.MTF_RESHAPE_SLICE, "alltoall": mtf.MTF_RESHAPE_ALLTOALL}


@pytest.mark.parametrize("mesh_dims", [[("a", 2)], [("a", 2), ("b", 3)], [("a", 2), ("b", 2), ("c", 2)]])
def test_reshape_plan_matches_oracle_lowering(mesh_dims):
    dims = [("p", 12), ("q", 6), ("r", 12)]
    out_names = ["p2", "z", "r"]
    x = NT(dims, si.small_integers(5, "x", [12, 6, 12]))
    n_legal = 0
    for rules in chooser.enumerate_layouts(mesh_dims, ["p", "q", "r", "p2", "z"]):
        lay = mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules)
        olay = Layout(Mesh(mesh_dims), rules)
        try:
            olay.tensor_layout(dims)
            olay.tensor_layout([(n, s) for n, (_, s) in zip(out_names, dims)])
        except OracleError as e:
            with pytest.raises(mtf.MtfError) as err:
                mtf.mtf_reshape_plan(lay, dims, out_names)
            assert err.value.code == e.code
            continue
        ops = LoweredOps(olay)
        ops.reshape(ops.lower(x), out_names)
        want_pat, want_rec = [0] * len(mesh_dims), [0] * len(mesh_dims)
        for j, pat, rec in ops.reshape_log:
            want_pat[j], want_rec[j] = PATTERN[pat], rec
        assert mtf.mtf_reshape_plan(lay, dims, out_names) == (want_pat, want_rec), rules
        n_legal += 1
    assert n_legal >= 8


def fc(b, d_io, d_h):
    x, w, v, h = [("batch", b), ("io", d_io)], [("io", d_io), ("hidden", d_h)], [("hidden", d_h), ("io", d_io)], [("batch", b), ("hidden", d_h)]
    return [(x, w, h), (h, v, x), (x, v, h), (h, x, v), (x, h, w), (h, w, x)]


@pytest.mark.parametrize("mesh_dims,b,d_io,d_h,cw", [([("all", 4)], 64, 8, 16, 4.0), ([("all", 4)], 16, 8, 64, 4.0), ([("rows", 2), ("cols", 4)], 32, 8, 32, 1.0),
                                                      ([("rows", 2), ("cols", 4)], 32, 8, 32, 0.0), ([("a", 2), ("b", 2), ("c", 2)], 16, 16, 16, 2.0),
                                                      ([("rows", 3), ("cols", 2)], 12, 6, 10, 1.5)])
def test_layout_search_matches_oracle_search(mesh_dims, b, d_io, d_h, cw):
    names = ["batch", "hidden", "io"]
    es = fc(b, d_io, d_h)
    want_rules, want_cost, want_foot = chooser.choose_layout(mesh_dims, names, [([i0, i1], [n for n, _ in o]) for i0, i1, o in es], cw)
    got = mtf.mtf_layout_search(mtf.mtf_mesh_create(mesh_dims), [tuple(mtf.desc(d, "bf16") for d in e) for e in es], names, cw)
    assert got == (want_rules, want_cost, want_foot)


def test_layout_search_transformer_dims_pick_the_paper_s_layout():
    # the Transformer feed-forward and attention projections on a 1-d mesh: with a small batch the cheapest
    # legal layout splits the model dimensions (d_ff, heads) as in Section 9
    B, L, D, F, H, K = 2, 64, 256, 2048, 16, 64
    act, hid = [("batch", B), ("length", L), ("d_model", D)], [("batch", B), ("length", L), ("d_ff", F)]
    w, v = [("d_model", D), ("d_ff", F)], [("d_ff", F), ("d_model", D)]
    q, wq, wo = [("batch", B), ("length", L), ("heads", H), ("d_k", K)], [("d_model", D), ("heads", H), ("d_k", K)], [("heads", H), ("d_k", K), ("d_model", D)]
    es = [(act, w, hid), (hid, v, act), (act, wq, q), (q, wo, act)]
    rules, _, _ = mtf.mtf_layout_search(mtf.mtf_mesh_create([("all", 8)]), [tuple(mtf.desc(d, "bf16") for d in e) for e in es], ["batch", "d_ff", "heads"], 1.0)
    assert rules == [("d_ff", "all"), ("heads", "all")]


def test_update_argument_checks():
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 2)]), [("d_ff", "all")])
    g, w = mtf.desc([("d_model", 4), ("d_ff", 8)], "f32"), mtf.desc([("d_model", 4), ("d_ff", 8)], "f32")
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_update(lay, g, w, None, None, 0.1)           # no data pointers
    assert e.value.code == "MTF_ERR_INVALID_ARG"


def test_tensor_core_plans_need_slices_that_start_on_16_byte_boundaries():
    # a tensor-map copy must start on a 16-byte boundary along the contiguous dimension: an operand whose
    # N dimension is contiguous and split into slices of 500 bf16 elements (1000 bytes) cannot be fed to the
    # tensor-core kernel slice by slice; the planner sends it to the generic kernel instead (and takes
    # the tensor cores again when the slices are multiples of 8 elements)
    h, o = mtf.desc([("tok", 144), ("d", 128)], "bf16"), None
    for vocab, want in ((1000, mtf.MTF_KERNEL_SIMT), (1024, mtf.MTF_KERNEL_TCGEN05)):
        lay = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 2)]), [("vocab", "all")])
        dlg = mtf.desc([("tok", 144), ("vocab", vocab)], "bf16")
        plan = mtf.mtf_einsum_plan(lay, [h, dlg], mtf.desc([("d", 128), ("vocab", vocab)], "f32"))
        assert mtf.mtf_plan_info(plan)["kernel_kind"] == want, vocab
        # the same with the split dimension on the M side (operands exchanged by the planner)
        plan = mtf.mtf_einsum_plan(lay, [dlg, h], mtf.desc([("vocab", vocab), ("d", 128)], "f32"))
        assert mtf.mtf_plan_info(plan)["kernel_kind"] == want, vocab
