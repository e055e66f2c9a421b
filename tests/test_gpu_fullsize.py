"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration the
bench times (planner's choices, C ABI).

Gate: stage-wise (stagewise.py) - every launch of the block against the exact fp64 oracle of that
launch, evaluated on the inputs the GPU launch actually read, at 1e-2 in the parity metric, on SAMPLED
outputs the oracle can compute one by one:
  * rows of sampled tokens (always the first and last token of every slice along a split dimension)
    for everything that has a token dimension;
  * whole (batch, head) pairs for the attention core (corners of every slice included);
  * columns of sampled hidden units / (head, d_k) pairs / d_model columns for the parameter
    gradients, each summed over ALL tokens, so the cross-slice sums are exercised end to end.
The elements that are not sampled are covered by comparing every layout's outputs with those of the
un-split mesh [1] (GPU against GPU, all elements).
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import TOL, ffn_inputs
from stagewise import run_attention_stagewise, run_decoder_stagewise, run_ffn_stagewise

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


def layout(mtf, mesh_dims, rules):
    return mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules)


def slice_edges(extent, nsplit):
    t = extent // nsplit
    return sorted({c * t for c in range(nsplit)} | {(c + 1) * t - 1 for c in range(nsplit)})


def device_errors(g, r):
    """(parity metric, rms error) of two device tensors, computed on the device in fp64 (the tensors
    of the largest configuration would not fit a host array of doubles comfortably)."""
    import torch
    g, r = g.double().flatten(), r.double().flatten()
    rms_r = r.pow(2).mean().sqrt().clamp_min(1e-300)
    d = (g - r).abs()
    par = (d / torch.maximum(r.abs(), rms_r)).max()
    rms = d.pow(2).sum().sqrt() / r.pow(2).sum().sqrt().clamp_min(1e-300)
    return float(par), float(rms)


def cross_layout(res, base, keys, what, elem_gate=True):
    """Every element of every output against the un-split run (same arithmetic, other tile boundaries
    and summation order): a one-ulp flip of a stored bf16 value is the largest legitimate difference."""
    for k in keys:
        par, rms = device_errors(res[k], base[k])
        assert rms <= 2e-3, (what, k, rms)
        if elem_gate:
            assert par <= TOL["bf16"], (what, k, par)


FFN_CASES = {
    "config2": dict(batch=32, length=256, d_model=1024, d_ff=4096, nsplit=8,
                    layouts=[([("all", 1)], []), ([("all", 8)], [("batch", "all")]), ([("all", 8)], [("d_ff", "all")])]),
    "target": dict(batch=32, length=256, d_model=1024, d_ff=8192, nsplit=8,
                   layouts=[([("all", 1)], []), ([("all", 8)], [("d_ff", "all")]), ([("all", 8)], [("batch", "all")]),
                            ([("rows", 2), ("cols", 4)], [("batch", "rows"), ("d_ff", "cols")]),                                       # Section 8.3, two-dimensional
                            ([("rows", 2), ("cols", 2), ("planes", 2)], [("batch", "rows"), ("d_ff", "cols"), ("d_model", "planes")])]),  # Section 8.3, three-dimensional
    "config4": dict(batch=32, length=256, d_model=1024, d_ff=65536, nsplit=16,
                    layouts=[([("all", 1)], []), ([("all", 16)], [("d_ff", "all")])]),
}


@pytest.mark.parametrize("name", list(FFN_CASES))
def test_ffn_full_size_stagewise(mtf, name):
    c = FFN_CASES[name]
    B, L, D, F = c["batch"], c["length"], c["d_model"], c["d_ff"]
    T = B * L
    inp = ffn_inputs(0, [("batch", B), ("length", L)], D, F, "bf16", True)
    # sampled tokens: first / last token of every batch slice (8 ways) + seeded picks; sampled hidden
    # units: first / last of every d_ff slice + seeded picks
    tok_edges = [b * L for b in slice_edges(B, 8)[:3]] + [b * L + L - 1 for b in slice_edges(B, 8)[-3:]] + [0, T - 1]
    tok = si.sample_indices(0, "tokens", T, 6, must_include=tok_edges)
    hid_edges = slice_edges(F, c["nsplit"])
    hid = si.sample_indices(0, "hidden", F, 6, must_include=hid_edges[:4] + hid_edges[-4:] + hid_edges[len(hid_edges) // 2:len(hid_edges) // 2 + 2])
    base = None
    for mesh_dims, rules in c["layouts"]:
        errs, out = run_ffn_stagewise(mtf, layout(mtf, mesh_dims, rules), inp, "bf16", tok=tok, hid=hid, what=f"{name} {rules}")
        print(name, rules, {k: f"{e:.2e}" for k, e in errs.items()})
        if base is None:
            base = out
        else:
            cross_layout(out, base, list(base), f"{name} {rules}")


def attention_samples(B, L, H, K, b_split, h_split, seed=0):
    bs, hs = slice_edges(B, b_split), slice_edges(H, h_split)
    pairs = sorted({(bs[0], hs[0]), (bs[-1], hs[-1]), (bs[1], hs[-2]), (bs[-2], hs[1]), (bs[len(bs) // 2], hs[len(hs) // 2])})
    tok = si.sample_indices(seed, "att_tokens", B * L, 6, must_include=[0, B * L - 1] + [b * L for b in bs[1:4]] + [b * L + L - 1 for b in bs[-4:-1]])
    wcols = sorted({(hs[0], 0), (hs[-1], K - 1), (hs[1], K // 2), (hs[-2], 1), (hs[len(hs) // 2], K - 2)})
    return tok, pairs, wcols


def test_attention_config3_full_size_stagewise(mtf):
    from test_gpu_attention import attention_case
    B, L, D, H, K = 16, 512, 1024, 16, 64
    inp = attention_case(0, B, L, D, H, K)
    tok, pairs, wcols = attention_samples(B, L, H, K, 4, 4)
    base = None
    for tag, mesh_dims, rules in (("unsplit", [("all", 1)], []), ("4x4", [("rows", 4), ("cols", 4)], [("batch", "rows"), ("heads", "cols")])):
        errs, out = run_attention_stagewise(mtf, layout(mtf, mesh_dims, rules), inp, False, tok=tok, pairs=pairs, wcols=wcols, what=f"config3 {tag}")
        print("config3", tag, {k: f"{e:.2e}" for k, e in errs.items()})
        if base is None:
            base = out
        else:
            cross_layout(out, base, list(base), f"config3 {tag}")


# the six mesh / layout combinations of the decoder-layer sweep that name dimensions the mesh has
DECODER_SWEEP = {
    "unsplit": ([("all", 1)], []),
    "batch8": ([("all", 8)], [("batch", "all")]),
    "model8": ([("all", 8)], [("d_ff", "all"), ("heads", "all")]),
    "4x8-batch": ([("rows", 4), ("cols", 8)], [("batch", "rows")]),
    "4x8-model": ([("rows", 4), ("cols", 8)], [("d_ff", "cols"), ("heads", "cols")]),
    "4x8": ([("rows", 4), ("cols", 8)], [("batch", "rows"), ("d_ff", "cols"), ("heads", "cols")]),
}


def test_decoder_layer_config5_full_size_stagewise(mtf):
    import torch
    from test_gpu_attention import decoder_case
    B, L, D, H, K, F = 64, 256, 2048, 32, 64, 8192
    inp = decoder_case(0, B, L, D, H, K, F)
    tok, pairs, wcols = attention_samples(B, L, H, K, 8, 8)
    hid_edges = slice_edges(F, 8)
    hid = si.sample_indices(0, "dec_hidden", F, 4, must_include=hid_edges[:3] + hid_edges[-3:])
    dcols = si.sample_indices(0, "dec_dcols", D, 6, must_include=[0, D - 1])
    base = None
    for tag, (mesh_dims, rules) in DECODER_SWEEP.items():
        errs, res = run_decoder_stagewise(mtf, layout(mtf, mesh_dims, rules), inp, tok=tok, pairs=pairs, wcols=wcols, hid=hid, dcols=dcols,
                                          what=f"config5 {tag}", causal_hint=tag != "model8")
        print("config5", tag, {k: f"{e:.2e}" for k, e in errs.items()})
        if base is None:
            base = {k: t.clone() for k, t in res.items()}
        else:
            # dx and the parameter gradients follow relu decisions and bf16 stores that both runs take
            # in the same precision on the same values: tight again
            cross_layout(res, base, list(base), f"config5 {tag}", elem_gate=False)
        del res
        torch.cuda.empty_cache()
