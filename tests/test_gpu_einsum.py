"""GPU parity of single einsums against the fp64 oracle, through the C ABI: every operand
major-ness the tensor-core path takes, ragged sizes, batched (attention-shaped) contractions, both
ways of realising the group sum, the fused epilogue stages, reductions and the slice gather."""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import TOL, from_torch, parity_error, to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


def layout(mtf, mesh_dims, rules):
    return mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules)


def run_einsum(mtf, lay, in_dims, out_dims, dtype, out_dtype=None, force=(-1, -1), seed=5, epilogue=None):
    """Runs one einsum on the GPU and in the oracle.  ``epilogue``: dict with optional keys scale,
    relu, bias (dims), relu_mask (True), residual (True).  Returns (got, ref, plan info)."""
    import torch
    from oracle import NT, DenseOps
    out_dtype = out_dtype or dtype
    tdt = {"bf16": torch.bfloat16, "f32": torch.float32}
    ins = [si.normal(seed, f"in{q}", [s for _, s in d], dtype, 1.0 if q == 0 else float(np.sqrt(1.0 / max(1, min(s for _, s in d)))))
           for q, d in enumerate(in_dims)]
    dev = [to_torch(s) for s in ins]
    names = [mtf.named(t, [n for n, _ in d]) for t, d in zip(dev, in_dims)]
    out = torch.full([s for _, s in out_dims], float("nan"), dtype=tdt[out_dtype], device="cuda")
    N_out = mtf.named(out, [n for n, _ in out_dims])
    ep = None
    ops = DenseOps()
    ref = ops.einsum([NT(d, s.f64) for d, s in zip(in_dims, ins)], [n for n, _ in out_dims])
    keep = []
    if epilogue:
        kw = {"scale": epilogue.get("scale", 1.0), "relu": epilogue.get("relu", False)}
        ref = ops.scale(ref, kw["scale"])
        if "bias" in epilogue:
            bd = epilogue["bias"]
            b = si.normal(seed, "bias", [s for _, s in bd], "f32", 0.5)
            bt = to_torch(b)
            keep.append(bt)
            kw["bias"] = mtf.named(bt, [n for n, _ in bd])
            ref = ops.add(ref, NT(bd, b.f64))
        if kw["relu"]:
            ref = ops.relu(ref)
        if epilogue.get("relu_mask"):
            m = si.normal(seed, "mask", [s for _, s in out_dims], out_dtype)
            mt = to_torch(m)
            keep.append(mt)
            kw["relu_mask"] = mtf.named(mt, [n for n, _ in out_dims])
            ref = ops.mul(ref, ops.positive(NT(out_dims, m.f64)))
        if epilogue.get("residual"):
            r = si.normal(seed, "res", [s for _, s in out_dims], out_dtype)
            rt = to_torch(r)
            keep.append(rt)
            kw["residual"] = mtf.named(rt, [n for n, _ in out_dims])
            ref = ops.add(ref, NT(out_dims, r.f64))
        ep = mtf.Epilogue(**kw)
    mtf.mtf_plan_force(*force)
    try:
        plan = mtf.mtf_einsum_plan(lay, names, N_out, ep)
        info = mtf.mtf_plan_info(plan)
        nbytes = mtf.mtf_plan_workspace_bytes(plan)
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        mtf.mtf_einsum_exec(plan, names, N_out, ep, ws)
    finally:
        mtf.mtf_plan_force(-1, -1)
    mtf.mtf_device_status()
    return from_torch(out), ref.a, info


# A[i,k] / A[k,i] x B[k,j] / B[j,k]: the four operand major-ness combinations, sizes that are not
# multiples of the tile (M 300 = 2 tiles + 44, N 328 = 1 tile + 72, K 200 = 3 k-blocks + 8)
MAJORS = {
    "K-major x MN-major": ([("i", 300), ("k", 200)], [("k", 200), ("j", 328)]),
    "K-major x K-major": ([("i", 300), ("k", 200)], [("j", 328), ("k", 200)]),
    "MN-major x MN-major": ([("k", 200), ("i", 304)], [("k", 200), ("j", 328)]),
    "MN-major x K-major": ([("k", 200), ("i", 304)], [("j", 328), ("k", 200)]),
}


@pytest.mark.parametrize("name", list(MAJORS))
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
@pytest.mark.parametrize("kind", [1, 2], ids=["cta-pairs", "single-cta"])
def test_tensor_core_operand_majors(mtf, name, out_dtype, kind):
    a, b = MAJORS[name]
    out_dims = [a[0] if a[0][0] == "i" else a[1], b[1] if b[1][0] == "j" else b[0]]
    lay = layout(mtf, [("all", 1)], [])
    got, ref, info = run_einsum(mtf, lay, [a, b], out_dims, "bf16", out_dtype, force=(kind, -1))
    assert info["kernel_kind"] == mtf.MTF_KERNEL_TCGEN05
    assert parity_error(got, ref) <= TOL["bf16"]


# 256 x 512 pair tiles (kernel_kind 3 forces them; the launcher refuses shapes they cannot run):
# ragged M, several k-blocks with a remainder, every operand major-ness, both output types
WIDE = {
    "K-major x MN-major": ([("i", 300), ("k", 200)], [("k", 200), ("j", 1024)]),
    "K-major x K-major": ([("i", 300), ("k", 200)], [("j", 1024), ("k", 200)]),
    "MN-major x MN-major": ([("k", 200), ("i", 304)], [("k", 200), ("j", 1024)]),
    "MN-major x K-major": ([("k", 200), ("i", 304)], [("j", 1024), ("k", 200)]),
}


@pytest.mark.parametrize("name", list(WIDE))
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_wide_pair_tiles(mtf, name, out_dtype):
    a, b = WIDE[name]
    out_dims = [a[0] if a[0][0] == "i" else a[1], b[1] if b[1][0] == "j" else b[0]]
    got, ref, info = run_einsum(mtf, layout(mtf, [("all", 1)], []), [a, b], out_dims, "bf16", out_dtype, force=(3, -1))
    assert info["kernel_kind"] == mtf.MTF_KERNEL_TCGEN05
    assert parity_error(got, ref) <= TOL["bf16"]


@pytest.mark.parametrize("mesh_dims,rules", [([("all", 2)], [("j", "all")]), ([("all", 4)], [("k", "all")]),
                                             ([("a", 2), ("b", 2)], [("o", "a"), ("k", "b")])],
                         ids=["n-split", "k-split-chained", "m-and-k-split"])
def test_wide_pair_tiles_under_layouts(mtf, mesh_dims, rules):
    # several tiles per worker in sequence (single accumulator: each tile's epilogue must finish
    # before the next tile's first MMA), batch dim, split N (slices of 512) and chained group sums
    a, b = [("o", 4), ("i", 960), ("k", 512)], [("k", 512), ("j", 1024)]      # o and i merge into M = 3840
    k_split = any(t == "k" for t, _ in rules)       # (the workspace reduce mode has no wide tiles: ask for the chained one)
    got, ref, info = run_einsum(mtf, layout(mtf, mesh_dims, rules), [a, b], [("o", 4), ("i", 960), ("j", 1024)], "bf16",
                                force=(3, 1 if k_split else -1))
    assert parity_error(got, ref) <= TOL["bf16"]


def test_wide_pair_tiles_refuse_what_they_cannot_run(mtf):
    lay = layout(mtf, [("all", 1)], [])
    with pytest.raises(mtf.MtfError) as e:      # N is not a multiple of 512
        run_einsum(mtf, lay, [[("i", 512), ("k", 128)], [("k", 128), ("j", 768)]], [("i", 512), ("j", 768)], "bf16", force=(3, -1))
    assert e.value.code == "MTF_ERR_UNSUPPORTED"
    with pytest.raises(mtf.MtfError) as e:      # not a plain epilogue
        run_einsum(mtf, lay, [[("i", 512), ("k", 128)], [("k", 128), ("j", 1024)]], [("i", 512), ("j", 1024)], "bf16", force=(3, -1),
                   epilogue={"relu": True})
    assert e.value.code == "MTF_ERR_UNSUPPORTED"
    got, ref, _ = run_einsum(mtf, lay, [[("i", 512), ("k", 128)], [("k", 128), ("j", 1024)]], [("i", 512), ("j", 1024)], "bf16", force=(4, -1))
    assert parity_error(got, ref) <= TOL["bf16"]


def test_tensor_core_transposed_output_swaps_operands(mtf):
    # out[j, i]: the contiguous output dim comes from the first operand
    a, b = [("i", 256), ("k", 128)], [("k", 128), ("j", 192)]
    got, ref, info = run_einsum(mtf, layout(mtf, [("all", 1)], []), [a, b], [("j", 192), ("i", 256)], "bf16", force=(1, -1))
    assert parity_error(got, ref) <= TOL["bf16"]


SPLITS = [
    ([("all", 4)], [("i", "all")]),
    ([("all", 4)], [("j", "all")]),
    ([("all", 4)], [("k", "all")]),
    ([("a", 2), ("b", 2)], [("i", "a"), ("k", "b")]),
    ([("a", 2), ("b", 2), ("c", 2)], [("i", "a"), ("j", "b"), ("k", "c")]),
]


@pytest.mark.parametrize("mesh_dims,rules", SPLITS)
@pytest.mark.parametrize("mode", [1, 2], ids=["chained", "workspace"])
@pytest.mark.parametrize("kind", [1, 2], ids=["cta-pairs", "single-cta"])
def test_tensor_core_split_dims_and_group_sum(mtf, mesh_dims, rules, mode, kind):
    a, b = [("i", 512), ("k", 512)], [("k", 512), ("j", 384)]
    lay = layout(mtf, mesh_dims, rules)
    k_split = any(t == "k" for t, _ in rules)
    if mode == 2 and not k_split:
        with pytest.raises(mtf.MtfError) as e:
            run_einsum(mtf, lay, [a, b], [("i", 512), ("j", 384)], "bf16", force=(kind, 2))
        assert e.value.code == "MTF_ERR_UNSUPPORTED"
        return
    got, ref, info = run_einsum(mtf, lay, [a, b], [("i", 512), ("j", 384)], "bf16", "f32", force=(kind, mode if k_split else -1))
    assert info["reduce_mode"] == (mode if k_split else 0)
    assert info["group_size"] == (2 if k_split and len(mesh_dims) > 1 else (4 if k_split else 1))
    assert parity_error(got, ref) <= TOL["bf16"]


def test_workspace_and_chained_agree_with_unsplit(mtf):
    a, b = [("k", 2048), ("i", 256)], [("k", 2048), ("j", 256)]      # a gradient-shaped contraction
    out = [("i", 256), ("j", 256)]
    res = {}
    for tag, mesh_dims, rules, force in (("unsplit", [("all", 1)], [], (1, -1)), ("chained", [("all", 8)], [("k", "all")], (1, 1)),
                                         ("workspace", [("all", 8)], [("k", "all")], (1, 2)), ("auto", [("all", 8)], [("k", "all")], (-1, -1))):
        got, ref, info = run_einsum(mtf, layout(mtf, mesh_dims, rules), [a, b], out, "bf16", "f32", force=force)
        assert parity_error(got, ref) <= TOL["bf16"], tag
        res[tag] = (got, info)
    # one output tile: the planner spreads the slices over CTAs only when that takes enough k-blocks
    # off the critical path to pay for the fragments (K = 2048 does not, K = 16384 does)
    assert res["auto"][1]["reduce_mode"] == mtf.MTF_REDUCE_CHAINED
    big = mtf.mtf_einsum_plan(layout(mtf, [("all", 8)], [("k", "all")]), [mtf.desc([("k", 16384), ("i", 256)], "bf16"), mtf.desc([("k", 16384), ("j", 256)], "bf16")],
                              mtf.desc(out, "f32"))
    assert mtf.mtf_plan_info(big)["reduce_mode"] == mtf.MTF_REDUCE_WORKSPACE
    # fp32 sums in different orders: equal to rounding, and the deterministic modes repeat bit for bit
    assert np.abs(res["chained"][0] - res["unsplit"][0]).max() <= 1e-3 * np.abs(res["unsplit"][0]).max()
    again, _, _ = run_einsum(mtf, layout(mtf, [("all", 8)], [("k", "all")]), [a, b], out, "bf16", "f32", force=(1, 2))
    assert np.array_equal(again, res["workspace"][0])


def test_balanced_k_range_schedule(mtf):
    """96 output tiles on 74 CTA pairs leave a partly filled second wave; with the balanced schedule
    every worker takes an equal range of (tile, k-block) units and cut tiles are assembled from two
    fragments.  Checked against the oracle on sampled rows and against the default schedule everywhere."""
    import torch
    from oracle import NT, DenseOps
    M, N, K = 4096, 1536, 2048
    a, b = si.normal(21, "a", [M, K], "bf16"), si.normal(21, "b", [K, N], "bf16", K ** -0.5)
    bias = si.normal(21, "bias", [N], "f32", 0.5)
    at, bt, biast = to_torch(a), to_torch(b), to_torch(bias)
    lay = layout(mtf, [("all", 4)], [("k", "all")])
    outs = {}
    for tag, force in (("default", (1, -1)), ("balanced", (1, 3))):
        out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        ins, O = [mtf.named(at, ["i", "k"]), mtf.named(bt, ["k", "j"])], mtf.named(out, ["i", "j"])
        ep = mtf.Epilogue(relu=True, bias=mtf.named(biast, ["j"]))
        mtf.mtf_plan_force(*force)
        try:
            plan = mtf.mtf_einsum_plan(lay, ins, O, ep)
            nbytes = mtf.mtf_plan_workspace_bytes(plan)
            assert (nbytes > 0) == (tag == "balanced")
            ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
            mtf.mtf_einsum_exec(plan, ins, O, ep, ws)
        finally:
            mtf.mtf_plan_force(-1, -1)
        mtf.mtf_device_status()
        outs[tag] = from_torch(out)
    rows = si.sample_indices(21, "rows", M, 40, must_include=[0, 255, 256, M - 1])
    ops = DenseOps()
    ref = ops.relu(ops.add(ops.einsum([NT([("i", len(rows)), ("k", K)], a.f64[rows]), NT([("k", K), ("j", N)], b.f64)], ["i", "j"]),
                           NT([("j", N)], bias.f64))).a
    for tag in outs:
        assert parity_error(outs[tag][rows], ref) <= TOL["bf16"], tag
    assert parity_error(outs["balanced"], outs["default"]) <= TOL["bf16"]


EPILOGUES = [
    {"scale": 0.125},
    {"relu": True, "bias": [("j", 328)]},
    {"bias": [("i", 300)]},
    {"relu_mask": True},
    {"residual": True, "scale": 0.5},
    {"relu": True, "bias": [("j", 328)], "relu_mask": True, "residual": True, "scale": 2.0},
]


@pytest.mark.parametrize("ep", EPILOGUES, ids=lambda e: "+".join(sorted(e)))
@pytest.mark.parametrize("kind", [0, 1], ids=["simt", "tcgen05"])
def test_fused_epilogue_stages(mtf, ep, kind):
    a, b = MAJORS["K-major x MN-major"]
    got, ref, info = run_einsum(mtf, layout(mtf, [("all", 2)], [("k", "all")]), [a, b], [("i", 300), ("j", 328)], "bf16",
                                force=(kind, -1), epilogue=ep)
    assert info["kernel_kind"] == kind
    assert parity_error(got, ref) <= TOL["bf16"]


def test_fused_reduce_sum_output(mtf):
    """dbias-style second output: sum over the rows of the masked value, fused into the einsum."""
    import torch
    from oracle import NT, DenseOps
    ops = DenseOps()
    a_d, b_d, o_d = [("t", 300), ("d", 200)], [("f", 328), ("d", 200)], [("t", 300), ("f", 328)]
    a, b, m = si.normal(6, "a", [300, 200], "bf16"), si.normal(6, "b", [328, 200], "bf16", 200 ** -0.5), si.normal(6, "m", [300, 328], "bf16")
    val = ops.mul(ops.einsum([NT(a_d, a.f64), NT(b_d, b.f64)], ["t", "f"]), ops.positive(NT(o_d, m.f64)))
    want = ops.reduce_sum(val, ["f"]).a
    at, bt, mt = to_torch(a), to_torch(b), to_torch(m)
    for kind, mesh_dims, rules in ((0, [("all", 1)], []), (1, [("all", 1)], []), (1, [("all", 4)], [("t", "all")]), (1, [("all", 4)], [("d", "all")])):
        out = torch.empty(300, 328, dtype=torch.bfloat16, device="cuda")
        rs = torch.full((328,), 7.0, dtype=torch.float32, device="cuda")          # the library zeroes it
        ep = mtf.Epilogue(relu_mask=mtf.named(mt, ["t", "f"]), reduce_sum_out=mtf.named(rs, ["f"]))
        mtf.mtf_plan_force(kind, -1)
        try:
            mtf.mtf_einsum(layout(mtf, mesh_dims, rules), "t d, f d -> t f", [mtf.named(at, ["t", "d"]), mtf.named(bt, ["f", "d"])],
                           mtf.named(out, ["t", "f"]), ep)
        finally:
            mtf.mtf_plan_force(-1, -1)
        mtf.mtf_device_status()
        assert parity_error(from_torch(rs), want) <= 1e-3, (kind, rules)
        assert parity_error(from_torch(out), val.a) <= TOL["bf16"]


# attention-shaped contractions (reading of Section 9: batch b, length l, memory m, heads h, d_k k)
B_, L_, H_, K_, D_ = 4, 160, 4, 64, 256
ATT = {
    "q = x.wq": ([("batch", B_), ("length", L_), ("d_model", D_)], [("d_model", D_), ("heads", H_), ("d_k", K_)],
                 [("batch", B_), ("length", L_), ("heads", H_), ("d_k", K_)]),
    "logits = q.k": ([("batch", B_), ("length", L_), ("heads", H_), ("d_k", K_)], [("batch", B_), ("memory_length", L_), ("heads", H_), ("d_k", K_)],
                     [("batch", B_), ("heads", H_), ("length", L_), ("memory_length", L_)]),
    "o = P.v": ([("batch", B_), ("heads", H_), ("length", L_), ("memory_length", L_)], [("batch", B_), ("memory_length", L_), ("heads", H_), ("d_v", K_)],
                [("batch", B_), ("length", L_), ("heads", H_), ("d_v", K_)]),
    "dv = P^T.do": ([("batch", B_), ("heads", H_), ("length", L_), ("memory_length", L_)], [("batch", B_), ("length", L_), ("heads", H_), ("d_v", K_)],
                    [("batch", B_), ("memory_length", L_), ("heads", H_), ("d_v", K_)]),
    "y = o.wo": ([("batch", B_), ("length", L_), ("heads", H_), ("d_v", K_)], [("heads", H_), ("d_v", K_), ("d_model", D_)],
                 [("batch", B_), ("length", L_), ("d_model", D_)]),
    "dwq = x^T.dq": ([("batch", B_), ("length", L_), ("d_model", D_)], [("batch", B_), ("length", L_), ("heads", H_), ("d_k", K_)],
                     [("d_model", D_), ("heads", H_), ("d_k", K_)]),
    "dx = dq.wq^T": ([("batch", B_), ("length", L_), ("heads", H_), ("d_k", K_)], [("d_model", D_), ("heads", H_), ("d_k", K_)],
                     [("batch", B_), ("length", L_), ("d_model", D_)]),
}


@pytest.mark.parametrize("name", list(ATT))
@pytest.mark.parametrize("mesh_dims,rules", [([("all", 1)], []), ([("rows", 2), ("cols", 2)], [("batch", "rows"), ("heads", "cols")])],
                         ids=["unsplit", "batch-x-heads"])
def test_attention_shaped_einsums_on_tensor_cores(mtf, name, mesh_dims, rules):
    a, b, out = ATT[name]
    got, ref, info = run_einsum(mtf, layout(mtf, mesh_dims, rules), [a, b], out, "bf16", force=(1, -1))
    assert info["kernel_kind"] == mtf.MTF_KERNEL_TCGEN05
    assert parity_error(got, ref) <= TOL["bf16"]


def test_generic_kernel_handles_what_tensor_cores_do_not(mtf):
    lay = layout(mtf, [("a", 2), ("b", 2)], [("length", "a"), ("j", "b")])
    cases = [
        # split on the inner component of a merged group (length inside (batch, length))
        ([("batch", 2), ("length", 8), ("k", 16)], [("k", 16), ("j", 24)], [("batch", 2), ("length", 8), ("j", 24)]),
        # a reduced dimension that only one operand carries
        ([("i", 6), ("p", 3), ("k", 16)], [("k", 16), ("j", 24)], [("i", 6), ("j", 24)]),
        # outer product, no reduced dimension
        ([("i", 6)], [("j", 24)], [("i", 6), ("j", 24)]),
        # odd sizes
        ([("i", 7), ("k", 13)], [("k", 13), ("j", 10)], [("j", 10), ("i", 7)]),
    ]
    for a, b, out in cases:
        for dt in ("f32", "bf16"):
            got, ref, info = run_einsum(mtf, lay, [a, b], out, dt)
            assert info["kernel_kind"] == mtf.MTF_KERNEL_SIMT
            assert parity_error(got, ref) <= TOL[dt], (a, b, out, dt)


def test_reduce_sum_under_layouts(mtf):
    import torch
    x = si.normal(9, "rx", [48, 40], "f32")
    xt = to_torch(x)
    for mesh_dims, rules in (([("all", 4)], []), ([("all", 4)], [("batch", "all")]), ([("a", 2), ("b", 2)], [("batch", "a"), ("hidden", "b")])):
        lay = layout(mtf, mesh_dims, rules)
        for out_dims, want in (([("hidden", 40)], x.f64.sum(0)), ([("batch", 48)], x.f64.sum(1)), ([], x.f64.sum())):
            out = torch.empty([s for _, s in out_dims], dtype=torch.float32, device="cuda")
            mtf.mtf_reduce_sum(lay, mtf.named(xt, ["batch", "hidden"]), mtf.named(out, [n for n, _ in out_dims]))
            assert parity_error(from_torch(out), want) <= TOL["f32"]


def test_slice_gather_is_bit_exact(mtf):
    import torch
    from oracle import Layout, Mesh
    dims = [("batch", 4), ("hidden", 6), ("io", 8)]
    mesh_dims, rules = [("rows", 2), ("cols", 3), ("planes", 2)], [("batch", "rows"), ("hidden", "cols"), ("io", "planes")]
    lay = layout(mtf, mesh_dims, rules)
    olay = Layout(Mesh(mesh_dims), rules)
    n = 4 * 6 * 8
    for tdt in (torch.float32, torch.bfloat16):
        payload = torch.arange(n, dtype=torch.float32).reshape(4, 6, 8).to(tdt).cuda()     # element = own flat index (exact in bf16 up to 256)
        for p in range(12):
            offs, sizes = mtf.mtf_slice_map(lay, dims, p)
            out = torch.empty(sizes, dtype=tdt, device="cuda")
            mtf.mtf_slice_gather(lay, mtf.named(payload, [d for d, _ in dims]), p, out)
            want = olay.global_flat_indices(dims, p).astype(np.float64)
            assert np.array_equal(from_torch(out).reshape(-1), want), (p, tdt)


def test_independent_hint_gives_the_same_results(mtf):
    """Contractions launched with mtf_hint_independent() may start while the launch before them still runs and
    draw their tiles from a counter; the counters are handed out in turn and cleared by each launch.  A chain of
    such launches (longer than the number of counters, so that the fall-back to an ordinary launch is taken
    too), issued several times over, must give bit for bit what the same contractions give without the hint."""
    import torch
    lay = layout(mtf, [("all", 1)], [])
    shapes = [(1024, 768, 4096), (4096, 2048, 512), (512, 512, 8192), (2304, 1280, 1024), (8192, 1024, 256), (768, 3072, 2048), (256, 256, 1024)]
    probs = []
    for i, (M, N, K) in enumerate(shapes):
        a = to_torch(si.normal(40 + i, "ha", [M, K], "bf16"))
        b = to_torch(si.normal(40 + i, "hb", [K, N], "bf16", K ** -0.5))
        outs = [torch.zeros(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        probs.append((mtf.named(a, ["m%d" % i, "k%d" % i]), mtf.named(b, ["k%d" % i, "n%d" % i]), outs, ["m%d" % i, "n%d" % i], (a, b)))
    for A, B, outs, names, _ in probs:
        mtf.mtf_einsum(lay, None, [A, B], mtf.named(outs[0], names))
    mtf.mtf_device_status()
    for rep in range(3):
        for _, _, outs, _, _ in probs:
            outs[1].zero_()
        for A, B, outs, names, _ in probs:
            mtf.mtf_hint_independent()
            mtf.mtf_einsum(lay, None, [A, B], mtf.named(outs[1], names))
        mtf.mtf_device_status()
        for i, (_, _, outs, _, _) in enumerate(probs):
            assert torch.equal(outs[0], outs[1]), (rep, shapes[i])


def test_independent_hint_is_used_up_by_the_next_einsum_whatever_runs_it(mtf):
    """The promise belongs to the next contraction only: an fp32 einsum on the generic kernel cannot honour it and must
    not pass it on to the launch after it, which here reads what the launch before it writes."""
    import torch
    lay = layout(mtf, [("all", 1)], [])
    a32 = to_torch(si.normal(61, "a32", [24, 40], "f32")); b32 = to_torch(si.normal(61, "b32", [40, 16], "f32"))
    c32 = torch.zeros(24, 16, dtype=torch.float32, device="cuda")
    M, N, K = 2048, 2048, 2048
    a = to_torch(si.normal(62, "a", [M, K], "bf16")); b = to_torch(si.normal(62, "b", [K, N], "bf16", K ** -0.5))
    mid = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda"); out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    w2 = to_torch(si.normal(63, "w2", [N, N], "bf16", N ** -0.5))
    def chain(hint):
        mtf.mtf_einsum(lay, None, [mtf.named(a, ["m", "k"]), mtf.named(b, ["k", "n"])], mtf.named(mid, ["m", "n"]))
        if hint:
            mtf.mtf_hint_independent()
        mtf.mtf_einsum(lay, None, [mtf.named(a32, ["i", "j"]), mtf.named(b32, ["j", "l"])], mtf.named(c32, ["i", "l"]))      # generic kernel: uses the hint up
        mtf.mtf_einsum(lay, None, [mtf.named(mid, ["m", "n"]), mtf.named(w2, ["n", "p"])], mtf.named(out, ["m", "p"]))       # depends on the first launch
        mtf.mtf_device_status()
        return out.clone()
    want = chain(False)
    for _ in range(3):
        mid.zero_(); out.zero_()
        assert torch.equal(chain(True), want)
