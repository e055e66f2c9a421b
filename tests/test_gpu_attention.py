"""GPU parity of softmax, layer normalisation, the attention block and the decoder layer against the
fp64 oracle, through the C ABI, under the Transformer layouts of Section 9."""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import TOL, end_to_end_report, from_torch, parity_error, rms_error, to_torch
from stagewise import PARAMS, run_attention_stagewise, run_decoder_stagewise

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


def layout(mtf, mesh_dims, rules):
    return mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules)


LAYOUTS = [
    ([("all", 1)], []),
    ([("all", 2)], [("batch", "all")]),
    ([("all", 4)], [("heads", "all"), ("d_ff", "all"), ("vocab", "all")]),
    ([("rows", 2), ("cols", 2)], [("batch", "rows"), ("heads", "cols"), ("d_ff", "cols")]),
]


def alloc(dims, dtype):
    import torch
    tdt = {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]
    return torch.full([s for _, s in dims], float("nan"), dtype=tdt, device="cuda")


# ---- softmax ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("causal", [False, True])
def test_softmax_forward_backward(mtf, causal):
    import torch
    dims = [("batch", 2), ("heads", 3), ("length", 40), ("memory_length", 40)]
    lg = si.normal(11, "lg", [2, 3, 40, 40], "f32", 2.0)
    dP = si.normal(11, "dP", [2, 3, 40, 40], "f32")
    x = lg.f64.copy()
    if causal:
        x = np.where(np.triu(np.ones((40, 40)), 1) > 0, -np.inf, x)
    e = np.exp(x - x.max(-1, keepdims=True))
    P = e / e.sum(-1, keepdims=True)
    names = [n for n, _ in dims]
    lay = layout(mtf, [("a", 2), ("b", 3)], [("batch", "a"), ("heads", "b")])
    w = alloc(dims, "bf16")
    mtf.mtf_softmax_forward(lay, mtf.named(to_torch(lg), names), causal, mtf.named(w, names))
    got = from_torch(w)
    assert parity_error(got, P) <= TOL["bf16"]
    if causal:
        iu = np.triu_indices(40, 1)
        assert (got[..., iu[0], iu[1]] == 0.0).all()
    # backward on the GPU's own (bf16) weights
    dlg = alloc(dims, "bf16")
    mtf.mtf_softmax_backward(lay, mtf.named(w, names), mtf.named(to_torch(dP), names), mtf.named(dlg, names))
    mtf.mtf_device_status()
    want = got * (dP.f64 - (dP.f64 * got).sum(-1, keepdims=True))
    assert parity_error(from_torch(dlg), want) <= TOL["bf16"]


# ---- einsum + softmax in one launch -------------------------------------------------------------------------

FUSED_SHAPES = [
    # (batch, heads, length, memory_length, d_k): a 128-row tile with a ragged tail, the single-CTA kernel
    (2, 2, 136, 136, 64),
    # CTA pairs, rows of three 64-column boxes (the two warps of a lane quarter own 2 and 1), 64 rows of the 256-row tile unused
    (2, 4, 192, 192, 64),
    # rows of 512: the wide pair tile (one accumulator)
    (1, 2, 512, 512, 32),
]


def _fused_case(seed, B, H, L, M, K):
    q = si.normal(seed, "q", [B, L, H, K], "bf16")
    kk = si.normal(seed, "kk", [B, M, H, K], "bf16")
    x = np.einsum("blhk,bmhk->bhlm", q.f64, kk.f64) * K ** -0.5
    return q, kk, x


@pytest.mark.parametrize("shape", FUSED_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("mesh_dims,rules", [([("all", 1)], []), ([("a", 2), ("b", 2)], [("batch", "a"), ("heads", "b")])][:2], ids=["one", "2x2"])
def test_einsum_softmax_one_launch(mtf, shape, causal, mesh_dims, rules):
    B, H, L, M, K = shape
    if B % 2 and len(mesh_dims) > 1:
        pytest.skip("batch of 1 cannot be split")
    q, kk, x = _fused_case(21, B, H, L, M, K)
    if causal:
        x = np.where(np.triu(np.ones((L, M)), 1) > 0, -np.inf, x)
    e = np.exp(x - x.max(-1, keepdims=True))
    P = e / e.sum(-1, keepdims=True)
    lay = layout(mtf, mesh_dims, rules)
    wdims = [("batch", B), ("heads", H), ("length", L), ("memory_length", M)]
    w = alloc(wdims, "bf16")
    n0 = mtf.mtf_launch_count()
    mtf.mtf_einsum_softmax(lay, mtf.named(to_torch(q), ["batch", "length", "heads", "d_k"]), mtf.named(to_torch(kk), ["batch", "memory_length", "heads", "d_k"]),
                           K ** -0.5, causal, mtf.named(w, [n for n, _ in wdims]))
    assert mtf.mtf_launch_count() - n0 == 1
    mtf.mtf_device_status()
    got = from_torch(w)
    assert parity_error(got, P) <= TOL["bf16"]
    if causal:
        iu = np.triu_indices(L, 1)
        assert (got[..., iu[0], iu[1]] == 0.0).all()
    assert np.abs(got.sum(-1) - 1.0).max() <= 2e-2          # rows of bf16 weights still sum to 1 within rounding


@pytest.mark.parametrize("shape", FUSED_SHAPES[1:], ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("causal", [False, True])
def test_einsum_softmax_backward_one_launch(mtf, shape, causal):
    B, H, L, M, V = shape
    do = si.normal(22, "do", [B, L, H, V], "bf16")
    vv = si.normal(22, "vv", [B, M, H, V], "bf16")
    lg = si.normal(22, "lg", [B, H, L, M], "f32", 2.0).f64
    if causal:
        lg = np.where(np.triu(np.ones((L, M)), 1) > 0, -np.inf, lg)
    e = np.exp(lg - lg.max(-1, keepdims=True))
    P = si.store(e / e.sum(-1, keepdims=True), "bf16")       # the weights as the forward pass keeps them
    dP = np.einsum("blhv,bmhv->bhlm", do.f64, vv.f64)
    want = P.f64 * (dP - (dP * P.f64).sum(-1, keepdims=True))
    lay = layout(mtf, [("a", 2)], [("heads", "a")])
    wdims = [("batch", B), ("heads", H), ("length", L), ("memory_length", M)]
    names = [n for n, _ in wdims]
    dlg = alloc(wdims, "bf16")
    n0 = mtf.mtf_launch_count()
    mtf.mtf_einsum_softmax_backward(lay, mtf.named(to_torch(do), ["batch", "length", "heads", "d_v"]),
                                    mtf.named(to_torch(vv), ["batch", "memory_length", "heads", "d_v"]), mtf.named(to_torch(P), names),
                                    mtf.named(dlg, names))
    assert mtf.mtf_launch_count() - n0 == 1
    mtf.mtf_device_status()
    assert parity_error(from_torch(dlg), want) <= TOL["bf16"]


def test_einsum_softmax_refuses_rows_that_do_not_fit(mtf):
    lay = layout(mtf, [("all", 1)], [])
    q, kk, _ = _fused_case(23, 1, 1, 64, 640, 64)             # 640 columns: more than a tile
    w = alloc([("batch", 1), ("heads", 1), ("length", 64), ("memory_length", 640)], "bf16")
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_softmax(lay, mtf.named(to_torch(q), ["batch", "length", "heads", "d_k"]), mtf.named(to_torch(kk), ["batch", "memory_length", "heads", "d_k"]),
                               0.125, False, mtf.named(w, ["batch", "heads", "length", "memory_length"]))
    assert e.value.code == "MTF_ERR_UNSUPPORTED"
    lay2 = layout(mtf, [("all", 2)], [("memory_length", "all")])      # rows split over processors
    q, kk, _ = _fused_case(23, 1, 1, 64, 128, 64)
    w = alloc([("batch", 1), ("heads", 1), ("length", 64), ("memory_length", 128)], "bf16")
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_einsum_softmax(lay2, mtf.named(to_torch(q), ["batch", "length", "heads", "d_k"]), mtf.named(to_torch(kk), ["batch", "memory_length", "heads", "d_k"]),
                               0.125, False, mtf.named(w, ["batch", "heads", "length", "memory_length"]))
    assert e.value.code == "MTF_ERR_UNSUPPORTED"


# ---- layer norm --------------------------------------------------------------------------------------------

# 136: the kernels that re-read the row per pass; 256..2048: rows kept in registers (2048: partial
# parameter sums in shared-memory strips); 50 rows per batch entry leave the last block ragged
@pytest.mark.parametrize("D", [136, 256, 512, 1024, 2048, 4096])
def test_layernorm_forward_backward(mtf, D):
    import torch
    from oracle import NT, DenseOps, blocks
    ops = DenseOps()
    dims = [("batch", 3), ("length", 50), ("d_model", D)]
    names = [n for n, _ in dims]
    x = si.normal(12, "x", [3, 50, D], "bf16", 2.0, 0.5)
    dy = si.normal(12, "dy", [3, 50, D], "bf16")
    res = si.normal(12, "res", [3, 50, D], "bf16")
    gamma = si.normal(12, "g", [D], "f32", 0.1, 1.0)
    beta = si.normal(12, "b", [D], "f32", 0.1)
    eps = 1e-6
    f = blocks.layernorm_forward(ops, NT(dims, x.f64), NT(dims[2:], gamma.f64), NT(dims[2:], beta.f64), eps)
    g = blocks.layernorm_backward(ops, NT(dims[2:], gamma.f64), f, NT(dims, dy.f64))
    lay = layout(mtf, [("all", 3)], [("batch", "all")])
    xt, dyt, rt, gt, bt = to_torch(x), to_torch(dy), to_torch(res), to_torch(gamma), to_torch(beta)
    y, dx = alloc(dims, "bf16"), alloc(dims, "bf16")
    stats = torch.empty(3, 50, 2, dtype=torch.float32, device="cuda")
    dg, db = alloc(dims[2:], "f32"), alloc(dims[2:], "f32")
    N = mtf.named
    mtf.mtf_layernorm_forward(lay, N(xt, names), N(gt, names[2:]), N(bt, names[2:]), eps, N(y, names), N(stats, ["batch", "length", "stat"]))
    mtf.mtf_layernorm_backward(lay, N(dyt, names), N(xt, names), N(stats, ["batch", "length", "stat"]), N(gt, names[2:]), N(rt, names),
                               N(dx, names), N(dg, names[2:]), N(db, names[2:]))
    mtf.mtf_device_status()
    # with a workspace the two column sums are added in a fixed order: the same values, bit for bit on every run
    nbytes = mtf.mtf_layernorm_workspace_bytes(D)
    if nbytes:
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        runs = []
        for _ in range(3):
            dg2, db2, dx2 = alloc(dims[2:], "f32"), alloc(dims[2:], "f32"), alloc(dims, "bf16")
            mtf.mtf_layernorm_backward(lay, N(dyt, names), N(xt, names), N(stats, ["batch", "length", "stat"]), N(gt, names[2:]), N(rt, names),
                                       N(dx2, names), N(dg2, names[2:]), N(db2, names[2:]), ws)
            mtf.mtf_device_status()
            runs.append((dg2, db2))
            assert torch.equal(dx2, dx)
        assert all(torch.equal(runs[0][0], r[0]) and torch.equal(runs[0][1], r[1]) for r in runs[1:])
        assert parity_error(from_torch(runs[0][0]), g["dgamma"].a) <= 1e-3 and parity_error(from_torch(runs[0][1]), g["dbeta"].a) <= 1e-3
    else:
        assert D in (136, 4096)          # these row lengths take the kernels without a fixed-order finish
    assert parity_error(from_torch(y), f["y"].a) <= TOL["bf16"]
    assert parity_error(from_torch(dx), g["dx"].a + res.f64) <= TOL["bf16"]
    assert parity_error(from_torch(dg), g["dgamma"].a) <= 1e-3
    assert parity_error(from_torch(db), g["dbeta"].a) <= 1e-3
    st = from_torch(stats)
    np.testing.assert_allclose(st[..., 0], x.f64.mean(-1), rtol=1e-4, atol=1e-5)
    np.testing.assert_allclose(st[..., 1], 1.0 / np.sqrt(x.f64.var(-1) + eps), rtol=1e-4)


# ---- attention ----------------------------------------------------------------------------------------------

def attention_case(seed, B, L, D, H, K):
    dims = {"x": [("batch", B), ("length", L), ("d_model", D)], "wq": [("d_model", D), ("heads", H), ("d_k", K)],
            "wk": [("d_model", D), ("heads", H), ("d_k", K)], "wv": [("d_model", D), ("heads", H), ("d_v", K)],
            "wo": [("heads", H), ("d_v", K), ("d_model", D)], "dy": [("batch", B), ("length", L), ("d_model", D)]}
    scale = {"x": 1.0, "dy": 1.0, "wq": D ** -0.5, "wk": D ** -0.5, "wv": D ** -0.5, "wo": (H * K) ** -0.5}
    return {k: (d, si.normal(seed, k, [s for _, s in d], "bf16", scale[k])) for k, d in dims.items()}


def run_attention_oracle(inp, causal, store_dtype):
    from oracle import NT, DenseOps, blocks, rounding
    ops = DenseOps()
    store = rounding.make_store(ops, store_dtype)
    T = {k: NT(d, s.f64) for k, (d, s) in inp.items()}
    L = T["x"].dims[1][1]
    mask = blocks.causal_mask(L) if causal else None
    f = blocks.attention_forward(ops, T["x"], T["wq"], T["wk"], T["wv"], T["wo"], mask, store)
    g = blocks.attention_backward(ops, T["x"], T["wq"], T["wk"], T["wv"], T["wo"], f, T["dy"], store)
    return {"y": f["y"].a, "P": f["P"].a, "o": f["o"].a, "q": f["q"].a, "dx": g["dx"].a, "dwq": g["dwq"].a, "dwk": g["dwk"].a,
            "dwv": g["dwv"].a, "dwo": g["dwo"].a}


@pytest.mark.parametrize("mesh_dims,rules", LAYOUTS)
@pytest.mark.parametrize("causal", [False, True])
def test_attention_block(mtf, mesh_dims, rules, causal):
    # length 136 = one 128-row tile + 8; d_k = d_v = 64 as in the paper-sized configurations.
    # Gate: every launch of the block, every element, against the exact oracle of that launch.
    inp = attention_case(13, 4, 136, 256, 4, 64)
    _, out = run_attention_stagewise(mtf, layout(mtf, mesh_dims, rules), inp, causal)
    ref = run_attention_oracle(inp, causal, None)
    end_to_end_report({k: from_torch(out[k]) for k in ref}, ref, f"attention causal={causal}")


def test_attention_small_head_dims(mtf):
    inp = attention_case(14, 2, 40, 64, 2, 32)            # d_k = 32: half a k-block, N tiles of 64 half used
    _, out = run_attention_stagewise(mtf, layout(mtf, [("all", 2)], [("heads", "all")]), inp, True)
    ref = run_attention_oracle(inp, True, None)
    end_to_end_report({k: from_torch(out[k]) for k in ref}, ref, "attention d_k=32")


@pytest.mark.parametrize("length", [128, 256, 384, 512])
@pytest.mark.parametrize("causal", [False, True, "unhinted"], ids=["full", "causal", "causal-unhinted"])
def test_attention_core_one_launch(mtf, length, causal):
    # d_k = d_v = 64 and rows of whole 128-key blocks up to 512: logits, softmax, the stored weights and
    # weights . v are one launch.  Every element of every stage against the exact oracle of that stage.
    inp = attention_case(13, 2, length, 256, 4, 64)
    lay = layout(mtf, [("rows", 2), ("cols", 2)], [("batch", "rows"), ("heads", "cols")])
    n0 = mtf.mtf_launch_count()
    # ("unhinted": causal weights, but the backward call is not told: it walks the all-zero blocks too)
    run_attention_stagewise(mtf, lay, inp, bool(causal), what=f"attention core L={length} causal={causal}", causal_hint=causal is True)
    # projections (1) + core (1) + output (1) forward; the backward's launches do not depend on the length
    assert mtf.mtf_launch_count() - n0 <= 12


@pytest.mark.parametrize("causal", [False, True])
def test_attention_core_many_tiles_per_block(mtf, causal):
    # more (pair, tile) items than the device has SMs: every thread block walks a range of query tiles that crosses
    # from one (batch, head) pair into the next (keys and values reloaded in mid-range); sampled pairs and tokens
    import seeded_inputs as si
    B, L, D, H, K = 6, 384, 256, 12, 64                      # 72 pairs x 3 tiles = 216 items
    inp = attention_case(17, B, L, D, H, K)
    pairs = sorted({(0, 0), (B - 1, H - 1), (2, 5), (3, 7), (4, 1), (1, 11)})
    tok = si.sample_indices(17, "core_tokens", B * L, 6, must_include=[0, B * L - 1, L - 1, L])
    wcols = [(0, 0), (H - 1, K - 1), (5, 31)]
    run_attention_stagewise(mtf, layout(mtf, [("all", 1)], []), inp, causal, tok=tok, pairs=pairs, wcols=wcols, what=f"attention core ranges causal={causal}")


@pytest.mark.parametrize("causal", [False, True])
def test_attention_core_many_pairs_per_block(mtf, causal):
    # more (batch, head) pairs than the device has SMs: a thread block of the backward core walks several pairs, with an
    # odd number of steps per pass when the weights are causal (rows of 256: blocks (0,0), (0,1), (1,1))
    import seeded_inputs as si
    B, L, D, H, K = 20, 256, 128, 16, 64                      # 320 pairs
    inp = attention_case(19, B, L, D, H, K)
    pairs = sorted({(0, 0), (B - 1, H - 1), (9, 3), (9, 4), (10, 15), (17, 8)})      # first, last and pairs a block reaches second or third
    tok = si.sample_indices(19, "pairs_tokens", B * L, 6, must_include=[0, B * L - 1, L - 1, L])
    wcols = [(0, 0), (H - 1, K - 1), (7, 31)]
    run_attention_stagewise(mtf, layout(mtf, [("all", 1)], []), inp, causal, tok=tok, pairs=pairs, wcols=wcols, what=f"attention core pairs causal={causal}")


# ---- decoder layer -------------------------------------------------------------------------------------------

def decoder_case(seed, B, L, D, H, K, F):
    inp = attention_case(seed, B, L, D, H, K)
    inp["dout"] = inp.pop("dy")
    inp["w"] = ([("d_model", D), ("d_ff", F)], si.normal(seed, "w", [D, F], "bf16", D ** -0.5))
    inp["v"] = ([("d_ff", F), ("d_model", D)], si.normal(seed, "v", [F, D], "bf16", F ** -0.5))
    inp["bias"] = ([("d_ff", F)], si.normal(seed, "bias", [F], "f32", 0.1))
    for n, shift in (("ln1_gamma", 1.0), ("ln1_beta", 0.0), ("ln2_gamma", 1.0), ("ln2_beta", 0.0)):
        inp[n] = ([("d_model", D)], si.normal(seed, n, [D], "f32", 0.1, shift))
    return inp


ORACLE_NAME = {"ln1_gamma": "g1", "ln1_beta": "b1", "ln2_gamma": "g2", "ln2_beta": "b2"}
GRAD_OF = {"wq": "dwq", "wk": "dwk", "wv": "dwv", "wo": "dwo", "ln1_gamma": "dg1", "ln1_beta": "db1", "w": "dw", "bias": "dbias", "v": "dv",
           "ln2_gamma": "dg2", "ln2_beta": "db2"}


def run_decoder_oracle(inp, store_dtype):
    from oracle import NT, DenseOps, blocks, rounding
    ops = DenseOps()
    store = rounding.make_store(ops, store_dtype)
    T = {k: NT(d, s.f64) for k, (d, s) in inp.items()}
    p = {ORACLE_NAME.get(k, k): T[k] for k in PARAMS}
    mask = blocks.causal_mask(T["x"].dims[1][1])
    f = blocks.decoder_layer_forward(ops, T["x"], p, mask, 1e-6, store)
    g = blocks.decoder_layer_backward(ops, T["x"], p, f, T["dout"], store)
    out = {"out": f["out"].a, "dx": g["dx"].a}
    for k in PARAMS:
        out["d_" + k] = g[GRAD_OF[k]].a
    hp = f["ffn"]["hp"].a
    return out, float(np.abs(hp).min() / np.sqrt(np.mean(hp * hp)))


@pytest.mark.parametrize("mesh_dims,rules", LAYOUTS)
def test_decoder_layer(mtf, mesh_dims, rules):
    # Gate: every launch of the layer (attention stages, both layer norms, feed-forward stages, forward
    # and backward), every element, against the exact oracle of that launch on the GPU's stored inputs.
    # End to end against exact mathematics the outputs are reported only: relu decisions taken on values
    # that the two sides hold one storage rounding apart move whole rows of the gradient stream, and
    # the layer-norm backward amplifies the storage rounding of the streams.
    inp = decoder_case(15, 4, 72, 128, 4, 32, 320)
    _, res = run_decoder_stagewise(mtf, layout(mtf, mesh_dims, rules), inp)
    ref, _ = run_decoder_oracle(inp, None)
    end_to_end_report({k: from_torch(res[k]) for k in ref}, ref, "decoder layer", rms_gate=None)
