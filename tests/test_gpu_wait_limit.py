"""The failure path of the bounded device-side waits, without faulting anything: a testing hook shortens the wait
limit to about a millisecond and withholds one signal (the "accumulator complete" signal of a launch's first tile),
so the epilogue's wait for it runs out.  The kernel must record the timeout, leave through its common teardown and
end normally; the host reads MTF_ERR_TIMEOUT; and an ordinary call right afterwards is correct."""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import TOL, from_torch, parity_error, to_torch

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_the_library_recovers():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as mtf
    from oracle import einsum_arrays
    a_dims, b_dims, out_dims = [("i", 128), ("k", 128)], [("k", 128), ("j", 128)], [("i", 128), ("j", 128)]      # one tile, two k-blocks
    a, b = si.normal(50, "a", [128, 128], "bf16"), si.normal(50, "b", [128, 128], "bf16", 128 ** -0.5)
    ins = [mtf.named(to_torch(a), ["i", "k"]), mtf.named(to_torch(b), ["k", "j"])]
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 1)]), [])
    out = torch.zeros(128, 128, dtype=torch.float32, device="cuda")
    mtf.mtf_plan_force(2, -1)                 # single-CTA tensor-core kernel
    try:
        mtf.mtf_device_status()
        mtf.mtf_debug_wait_test(2_000_000, True)      # ~1 ms at the boost clock, and the signal is withheld
        try:
            mtf.mtf_einsum(lay, None, ins, mtf.named(out, ["i", "j"]))
            with pytest.raises(mtf.MtfError) as e:
                mtf.mtf_device_status()
            assert e.value.code == "MTF_ERR_TIMEOUT"
        finally:
            mtf.mtf_debug_wait_test(0, False)
        mtf.mtf_device_status()                       # the status word was reset, the context is intact
        out.fill_(float("nan"))
        mtf.mtf_einsum(lay, None, ins, mtf.named(out, ["i", "j"]))
        mtf.mtf_device_status()
        ref = einsum_arrays([a_dims, b_dims], [a.f64, b.f64], out_dims)
        assert parity_error(from_torch(out), ref) <= TOL["bf16"]
    finally:
        mtf.mtf_plan_force(-1, -1)
