"""Shared helpers of the tests: moving seeded inputs to the device, the parity metric, and the
feed-forward parity routine used at several sizes."""
from __future__ import annotations

import numpy as np

import seeded_inputs as si


def to_torch(stored, device="cuda"):
    """seeded_inputs.Stored -> torch tensor with exactly those bytes."""
    import torch
    if stored.dtype == "bf16":
        t = torch.from_numpy(stored.bits.view(np.int16).copy()).view(torch.bfloat16)
    else:
        t = torch.from_numpy(stored.bits.copy())
    return t.to(device)


def from_torch(t) -> np.ndarray:
    """Device tensor -> fp64 numpy array (exact widening)."""
    import torch
    return t.detach().to("cpu").to(torch.float64).numpy()


def parity_error(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |g_i - r_i| / max(|r_i|, rms(r)): relative error that does not blow up at zeros."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), max(rms, 1e-300))
    return float(np.max(np.abs(got - ref) / den))


def rms_error(got, ref) -> float:
    """||g - r||_2 / ||r||_2: insensitive to isolated one-ulp differences, sensitive to anything systematic."""
    ref = np.asarray(ref, dtype=np.float64)
    d = np.asarray(got, dtype=np.float64) - ref
    return float(np.sqrt((d * d).sum()) / max(np.sqrt((ref * ref).sum()), 1e-300))


TOL = {"bf16": 1e-2, "f32": 1e-4}      # the parity metric a single launch is held to, against exact fp64 mathematics


class Guarded:
    """Device allocations with guard bands: every tensor handed out sits inside a larger buffer whose
    margins hold a sentinel byte pattern; ``check()`` asserts that no kernel wrote outside a tensor
    (a stand-in for a memory checker: NaN pre-fill catches unwritten elements, the bands catch writes
    that miss the tensor)."""
    MARGIN = 4096
    SENTINEL = 0xA5

    def __init__(self):
        self.items = []

    def empty(self, shape, dtype, fill=float("nan")):
        import torch
        tdt = {"bf16": torch.bfloat16, "f32": torch.float32, "u8": torch.uint8}[dtype] if isinstance(dtype, str) else dtype
        n = int(np.prod(shape)) if len(shape) else 1
        nbytes = n * torch.empty(0, dtype=tdt).element_size()
        padded = (nbytes + 255) // 256 * 256
        raw = torch.full((padded + 2 * self.MARGIN,), self.SENTINEL, dtype=torch.uint8, device="cuda")
        t = raw[self.MARGIN:self.MARGIN + nbytes].view(tdt).view(*shape)
        if fill is not None and tdt != torch.uint8:
            t.fill_(fill)
        self.items.append((raw, nbytes))
        return t

    def check(self):
        import torch
        for raw, nbytes in self.items:
            lo = raw[:self.MARGIN]
            hi = raw[self.MARGIN + (nbytes + 255) // 256 * 256:]
            tail = raw[self.MARGIN + nbytes:self.MARGIN + (nbytes + 255) // 256 * 256]
            for band in (lo, hi, tail):
                assert bool((band == self.SENTINEL).all()), "a kernel wrote outside a tensor (guard band overwritten)"


def ffn_inputs(seed, tok_dims, d_model, d_ff, dtype, with_bias=True, io_name="d_model", hidden_name="d_ff"):
    """The feed-forward workload: x ~ N(0,1), w ~ N(0,1/d_model), v ~ N(0,1/d_ff), bias ~ 0.1 N(0,1),
    dy ~ N(0,1).  Returns dict name -> (dims, Stored)."""
    tok_shape = [s for _, s in tok_dims]
    out = {
        "x": (list(tok_dims) + [(io_name, d_model)], si.normal(seed, "x", tok_shape + [d_model], dtype)),
        "w": ([(io_name, d_model), (hidden_name, d_ff)], si.normal(seed, "w", [d_model, d_ff], dtype, d_model ** -0.5)),
        "v": ([(hidden_name, d_ff), (io_name, d_model)], si.normal(seed, "v", [d_ff, d_model], dtype, d_ff ** -0.5)),
        "dy": (list(tok_dims) + [(io_name, d_model)], si.normal(seed, "dy", tok_shape + [d_model], dtype)),
    }
    if with_bias:
        out["bias"] = ([(hidden_name, d_ff)], si.normal(seed, "bias", [d_ff], "f32", 0.1))
    return out


def run_ffn_oracle(inp):
    """The whole block in exact fp64 mathematics on the same (rounded) inputs, nothing rounded in
    between: the end-to-end reference.  (The gate is stage-wise, see stagewise.py; end to end the
    storage rounding of h and dhp and single relu decisions taken on values within rounding of zero
    legitimately move outputs, so this comparison is reported and gated in the rms only.)"""
    from oracle import NT, DenseOps, blocks
    ops = DenseOps()
    T = {k: NT(d, s.f64) for k, (d, s) in inp.items()}
    f = blocks.ffn_forward(ops, T["x"], T["w"], T.get("bias"), T["v"])
    g = blocks.ffn_backward(ops, T["x"], T["w"], T["v"], f["h"], T["dy"])
    ref = {"h": f["h"].a, "y": f["y"].a, "dx": g["dx"].a, "dw": g["dw"].a, "dv": g["dv"].a}
    if "bias" in inp:
        ref["dbias"] = g["dbias"].a
    return ref


def end_to_end_report(got, ref, what, rms_gate=1e-2):
    """Parity metric and rms error of every output of a block against exact end-to-end mathematics.
    Printed; only the rms is gated (at the single-launch tolerance)."""
    rows = {k: (parity_error(got[k], ref[k]), rms_error(got[k], ref[k])) for k in ref}
    print(f"[end to end] {what}: " + ", ".join(f"{k} elem {e:.2e} rms {r:.2e}" for k, (e, r) in rows.items()))
    if rms_gate is not None:
        bad = {k: r for k, (_, r) in rows.items() if not r <= rms_gate}
        assert not bad, f"{what}: end-to-end rms error above {rms_gate}: {bad}"
    return rows


