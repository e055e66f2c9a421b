"""The entry point for callers that cannot allocate device memory (mtf_einsum_builtin_scratch).

Some users of this library are handed tensors but may not create device memory themselves: a
plug-in inside a host application that owns the allocator, a latency-critical loop where an
allocation's implicit device synchronisation is not acceptable, code that is replayed and must not
touch the allocator.  They cannot supply the workspace that mtf_einsum needs when the group sum over
the slices of a split contraction dimension goes through partial tiles.  The extra entry point runs
the same kernel on a fixed scratch array that is part of the library.  This test drives it through
the C ABI and compares its output with the regular entry point's, twice in a row because the
scratch array keeps the previous call's contents.

(File name chosen so that pytest collects it last: if it fails, every other test has already run.)
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import TOL, from_torch, parity_error, to_torch

pytestmark = pytest.mark.gpu


def test_builtin_scratch_matches_regular_entry_point_twice():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as mtf

    # a gradient-shaped contraction: the reduced dimension k is split over 8 virtual processors, so
    # the group sum runs through partial tiles in scratch memory (workspace mode)
    a_dims, b_dims, out_dims = [("k", 2048), ("i", 256)], [("k", 2048), ("j", 384)], [("i", 256), ("j", 384)]
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 8)]), [("k", "all")])
    mtf.mtf_plan_force(1, mtf.MTF_REDUCE_WORKSPACE)
    try:
        for call in range(2):
            a = si.normal(40 + call, "a", [2048, 256], "bf16")
            b = si.normal(40 + call, "b", [2048, 384], "bf16", 2048 ** -0.5)
            at, bt = to_torch(a), to_torch(b)
            ins = [mtf.named(at, ["k", "i"]), mtf.named(bt, ["k", "j"])]
            want = torch.full((256, 384), float("nan"), dtype=torch.float32, device="cuda")
            got = torch.full((256, 384), float("nan"), dtype=torch.float32, device="cuda")
            nbytes = mtf.mtf_einsum_workspace_bytes(lay, ins, mtf.named(want, ["i", "j"]))
            assert 0 < nbytes <= 32 << 20          # this shape does use scratch, and it fits the built-in array
            ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            mtf.mtf_einsum(lay, "k i, k j -> i j", ins, mtf.named(want, ["i", "j"]), None, ws)
            mtf.mtf_einsum_builtin_scratch(lay, "k i, k j -> i j", ins, mtf.named(got, ["i", "j"]))
            mtf.mtf_device_status()
            g, w = from_torch(got), from_torch(want)
            assert np.isfinite(g).all()
            # both entry points add the same partial tiles in the same (ascending processor) order
            assert parity_error(g, w) <= TOL["bf16"], call
            assert np.array_equal(g, w), call
            # and what they compute is the einsum: against the fp64 oracle on the same inputs
            from oracle import einsum_arrays
            ref = einsum_arrays([a_dims, b_dims], [a.f64, b.f64], out_dims)
            assert parity_error(g, ref) <= TOL["bf16"], call
        # arguments are validated on every call, as through the regular entry point: a relu mask of the
        # wrong shape handed in after a good call with the same stages is refused before any launch
        mask_ok = torch.ones(256, 384, dtype=torch.float32, device="cuda")
        mask_bad = torch.ones(128, 384, dtype=torch.float32, device="cuda")
        out = torch.empty(256, 384, dtype=torch.float32, device="cuda")
        mtf.mtf_einsum_builtin_scratch(lay, None, ins, mtf.named(out, ["i", "j"]), mtf.Epilogue(relu_mask=mtf.named(mask_ok, ["i", "j"])))
        mtf.mtf_device_status()
        assert np.array_equal(from_torch(out), from_torch(got))          # a mask of ones keeps everything
        n0 = mtf.mtf_launch_count()
        with pytest.raises(mtf.MtfError) as e:
            mtf.mtf_einsum_builtin_scratch(lay, None, ins, mtf.named(out, ["i", "j"]), mtf.Epilogue(relu_mask=mtf.named(mask_bad, ["i", "j"])))
        assert e.value.code in ("MTF_ERR_INVALID_ARG", "MTF_ERR_SIZE_MISMATCH")
        assert mtf.mtf_launch_count() == n0
        # a contraction whose partial tiles do not fit the built-in array is refused before any launch
        big_a, big_b = mtf.desc([("k", 8192), ("i", 4096)], "bf16"), mtf.desc([("k", 8192), ("j", 4096)], "bf16")
        n0 = mtf.mtf_launch_count()
        with pytest.raises(mtf.MtfError) as e:
            mtf.mtf_einsum_builtin_scratch(lay, None, [big_a, big_b], mtf.desc([("i", 4096), ("j", 4096)], "f32"))
        assert e.value.code == "MTF_ERR_WORKSPACE_TOO_SMALL"
        assert mtf.mtf_launch_count() == n0
    finally:
        mtf.mtf_plan_force(-1, -1)
