"""GPU parity of the feed-forward block (Section 8) against the fp64 oracle, through the C ABI.
Gate: every launch of the block against the exact oracle of that launch on the inputs the launch
read (stagewise.py), every element, at the single-launch tolerance; the end-to-end comparison with
exact mathematics is reported and held to that tolerance in the rms."""
import numpy as np
import pytest

from helpers import TOL, end_to_end_report, ffn_inputs, from_torch, run_ffn_oracle
from stagewise import run_ffn_stagewise

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


def make_layout(mtf, mesh_dims, rules):
    mesh = mtf.mtf_mesh_create(mesh_dims)
    return mtf.mtf_layout(mesh, rules)


def check_block(mtf, lay, inp, dtype, grad_dtype="f32"):
    errs, out = run_ffn_stagewise(mtf, lay, inp, dtype, grad_dtype)
    end_to_end_report({k: from_torch(t) for k, t in out.items()}, run_ffn_oracle(inp), "ffn", rms_gate=TOL[dtype])
    return errs


# ---- configuration 1: the fp32 toy of Section 8 on a 2x2 mesh ----------------------------------------

@pytest.mark.parametrize("with_bias", [False, True])
def test_config1_fp32_toy_mesh_2x2(mtf, with_bias):
    inp = ffn_inputs(0, [("batch", 8)], 64, 256, "f32", with_bias, io_name="io", hidden_name="hidden")
    lay = make_layout(mtf, [("rows", 2), ("cols", 2)], [("batch", "rows"), ("hidden", "cols")])
    check_block(mtf, lay, inp, "f32")


FP32_LAYOUTS = [
    ([("all", 4)], []),
    ([("all", 4)], [("batch", "all")]),
    ([("all", 4)], [("hidden", "all")]),
    ([("rows", 2), ("cols", 2)], [("batch", "rows"), ("hidden", "cols")]),
    ([("rows", 2), ("cols", 2), ("planes", 2)], [("batch", "rows"), ("hidden", "cols"), ("io", "planes")]),
    ([("rows", 2), ("cols", 3)], [("batch", "cols"), ("io", "rows")]),
]


@pytest.mark.parametrize("mesh_dims,rules", FP32_LAYOUTS)
def test_fp32_every_layout_of_the_example(mtf, mesh_dims, rules):
    inp = ffn_inputs(1, [("batch", 12)], 40, 72, "f32", True, io_name="io", hidden_name="hidden")
    check_block(mtf, make_layout(mtf, mesh_dims, rules), inp, "f32")


# ---- bf16 on the tensor-core path: several tiles, ragged tails, every layout family ------------------

BF16_LAYOUTS = [
    ([("all", 1)], []),
    ([("all", 8)], [("batch", "all")]),
    ([("all", 8)], [("d_ff", "all")]),
    ([("rows", 2), ("cols", 4)], [("batch", "rows"), ("d_ff", "cols")]),
    ([("all", 2)], [("d_model", "all")]),
]


@pytest.mark.parametrize("mesh_dims,rules", BF16_LAYOUTS)
@pytest.mark.parametrize("force", [(-1, -1), (1, 1), (2, 1), (0, -1)], ids=["auto", "tc-chained", "tc-single-cta", "simt"])
def test_bf16_ffn_layouts(mtf, mesh_dims, rules, force):
    # tokens 8 x 72 = 576 (4.5 row tiles), d_model 320 (5 k-blocks, 1.25 column tiles), d_ff 1088 (17 k-blocks)
    inp = ffn_inputs(2, [("batch", 8), ("length", 72)], 320, 1088, "bf16", True)
    mtf.mtf_plan_force(*force)
    try:
        check_block(mtf, make_layout(mtf, mesh_dims, rules), inp, "bf16")
    finally:
        mtf.mtf_plan_force(-1, -1)


def test_bf16_outputs_bf16_grads(mtf):
    inp = ffn_inputs(4, [("batch", 4), ("length", 64)], 256, 512, "bf16", True)
    check_block(mtf, make_layout(mtf, [("all", 4)], [("batch", "all")]), inp, "bf16", grad_dtype="bf16")


def test_column_sums_repeat_bit_for_bit(mtf):
    """dbias = sum over tokens of dhp rides in the dhp launch; with the block's workspace its per-row-group partial
    sums are finished in a fixed order, so - like every other output of the block - it is identical from run to run."""
    import torch
    inp = ffn_inputs(5, [("batch", 8), ("length", 72)], 320, 1088, "bf16", True)
    runs = []
    for _ in range(3):
        _, out = run_ffn_stagewise(mtf, make_layout(mtf, [("rows", 2), ("cols", 4)], [("batch", "rows"), ("d_ff", "cols")]), inp, "bf16")
        runs.append({k: t.clone() for k, t in out.items()})
    for r in runs[1:]:
        for k in runs[0]:
            assert torch.equal(runs[0][k], r[k]), k
