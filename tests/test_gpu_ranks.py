"""One mesh dimension across ranks, on ONE GPU: the ranks' local computations run one after the other
(independent launches, nothing waits on another rank), each under its rank-bound layout on its box of
every tensor, with collective hooks that only record which results the library wants summed.  The
test then adds the flagged partial results up itself (standing in for the all-reduce), glues the
split outputs together, and compares with the un-split run of the same block on the same GPU (that
run is held to the oracle stage by stage elsewhere).  Both ways the path shards are covered: batch
over ranks (the parameter gradients are summed: Algorithm 1 line 2) and the hidden / heads dimension
over ranks (y and dx are summed: Section 8.2), each combined with a second mesh dimension inside the rank."""
import numpy as np
import pytest

from helpers import TOL, ffn_inputs, to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


class Recorder:
    """Collective hooks that do nothing but remember what was asked to be summed."""

    def __init__(self, mtf):
        from paper_1811_02084_b200.binding import RANK_ALLREDUCE_FN, RANK_WAIT_FN
        self.started, self.waits = [], 0
        self.start_cb = RANK_ALLREDUCE_FN(lambda user, data, count, dtype, stream: self.started.append((int(data), int(count), int(dtype))) or 0)
        self.wait_cb = RANK_WAIT_FN(lambda user, stream: setattr(self, "waits", self.waits + 1) or 0)


def box_of(mtf, bound, t, dims):
    offs, sizes = mtf.mtf_rank_box(bound, dims)
    sl = tuple(slice(o, o + s) for o, s in zip(offs, sizes))
    return t[sl].contiguous(), [(n, s) for (n, _), s in zip(dims, sizes)], sl


def close(got, ref, what):
    import torch
    g, r = got.double(), ref.double()
    rms = float(r.pow(2).mean().sqrt())
    err = float(((g - r).abs() / torch.maximum(r.abs(), torch.tensor(rms, device=r.device, dtype=torch.float64))).max())
    assert err <= TOL["bf16"], (what, err)


@pytest.mark.parametrize("split", ["batch", "d_ff"])
def test_ffn_block_over_two_ranks(mtf, split):
    import torch
    B, L, D, F = 8, 64, 256, 1024
    inp = ffn_inputs(7, [("batch", B), ("length", L)], D, F, "bf16", True)
    dev = {k: to_torch(s) for k, (_, s) in inp.items()}
    dims = {k: d for k, (d, _) in inp.items()}
    dims.update({"h": dims["x"][:-1] + [("d_ff", F)], "y": dims["x"], "dx": dims["x"], "dw": dims["w"], "dv": dims["v"], "dbias": dims["bias"]})
    out_dtype = {"h": torch.bfloat16, "y": torch.float32, "dx": torch.float32, "dw": torch.float32, "dv": torch.float32, "dbias": torch.float32}
    mesh = [("ranks", 2), ("inner", 2)]
    rules = [("batch", "ranks"), ("d_ff", "inner")] if split == "batch" else [("d_ff", "ranks"), ("batch", "inner")]

    def run(lay, T, Dm):
        N = {k: mtf.named(T[k], [n for n, _ in Dm[k]]) for k in T}
        O = {k: torch.full([s for _, s in Dm[k]], float("nan"), dtype=out_dtype[k], device="cuda") for k in out_dtype}
        NO = {k: mtf.named(O[k], [n for n, _ in Dm[k]]) for k in O}
        ws = torch.empty(mtf.mtf_ffn_workspace_bytes(lay, N["x"], N["w"]), dtype=torch.uint8, device="cuda")
        mtf.mtf_ffn_forward(lay, N["x"], N["w"], N["bias"], N["v"], NO["h"], NO["y"], ws)
        mtf.mtf_ffn_backward(lay, N["x"], N["w"], N["v"], NO["h"], N["dy"], NO["dx"], NO["dw"], NO["dbias"], NO["dv"], ws)
        mtf.mtf_device_status()
        return O

    ref = run(mtf.mtf_layout(mtf.mtf_mesh_create([("all", 1)]), []), dev, dims)
    lay = mtf.mtf_layout(mtf.mtf_mesh_create(mesh), rules)
    total = {k: torch.zeros_like(v) for k, v in ref.items()}
    summed_names = None
    for rank in range(2):
        rec = Recorder(mtf)
        bound = mtf.mtf_layout_bind_ranks(lay, "ranks", 2, rank, rec)
        T, Dm, SL = {}, {}, {}
        for k in list(dev) + list(out_dtype):
            src = dev[k] if k in dev else ref[k]
            T[k], Dm[k], SL[k] = box_of(mtf, bound, src, dims[k])
        O = run(bound, {k: T[k] for k in dev}, Dm)
        ptr_name = {O[k].data_ptr(): k for k in O}
        names = sorted(ptr_name[p] for p, _, _ in rec.started)
        assert all(c == O[ptr_name[p]].numel() for p, c, _ in rec.started)
        assert rec.waits >= 2                                   # each block call waits before it returns
        summed_names = names if summed_names is None else summed_names
        assert names == summed_names
        for k in O:
            if k in names:
                total[k][SL[k]] += O[k]                         # the all-reduce: partial results add up
            else:
                total[k][SL[k]] = O[k]                          # a box of a split tensor, or a replica (written twice, identically)
    assert summed_names == (["dbias", "dv", "dw"] if split == "batch" else ["dx", "y"])
    for k in ref:
        close(total[k], ref[k], (split, k))


@pytest.mark.parametrize("split", ["batch", "heads"])
def test_attention_block_over_two_ranks(mtf, split):
    import torch
    from test_gpu_attention import attention_case
    B, L, D, H, K = 4, 72, 128, 4, 32
    inp = attention_case(8, B, L, D, H, K)
    dev = {k: to_torch(s) for k, (_, s) in inp.items()}
    dims = {k: d for k, (d, _) in inp.items()}
    m = "memory_length"
    dims.update({"q": [("batch", B), ("length", L), ("heads", H), ("d_k", K)], "kk": [("batch", B), (m, L), ("heads", H), ("d_k", K)],
                 "vv": [("batch", B), (m, L), ("heads", H), ("d_v", K)], "P": [("batch", B), ("heads", H), ("length", L), (m, L)],
                 "o": [("batch", B), ("length", L), ("heads", H), ("d_v", K)], "y": dims["x"], "dx": dims["x"],
                 "dwq": dims["wq"], "dwk": dims["wk"], "dwv": dims["wv"], "dwo": dims["wo"]})
    f32 = ("y", "dx", "dwq", "dwk", "dwv", "dwo")
    outs = ("q", "kk", "vv", "P", "o") + f32
    rules = [("batch", "ranks"), ("heads", "inner")] if split == "batch" else [("heads", "ranks"), ("batch", "inner")]

    def run(lay, T, Dm):
        N = {k: mtf.named(T[k], [n for n, _ in Dm[k]]) for k in T}
        O = {k: torch.full([s for _, s in Dm[k]], float("nan"), dtype=torch.float32 if k in f32 else torch.bfloat16, device="cuda") for k in outs}
        NO = {k: mtf.named(O[k], [n for n, _ in Dm[k]]) for k in O}
        ws = torch.empty(mtf.mtf_attention_workspace_bytes(lay, N["x"], N["wq"], N["wv"]), dtype=torch.uint8, device="cuda")
        mtf.mtf_attention_forward(lay, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], True, N["x"], NO["q"], NO["kk"], NO["vv"], NO["P"], NO["o"], NO["y"], ws)
        mtf.mtf_attention_backward(lay, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], NO["q"], NO["kk"], NO["vv"], NO["P"], NO["o"], N["dy"], N["dy"],
                                   NO["dx"], NO["dwq"], NO["dwk"], NO["dwv"], NO["dwo"], ws)
        mtf.mtf_device_status()
        return O

    # (x rides in y as a residual and dy in dx, as in the decoder layer: under a heads split rank 0 alone adds them)
    ref = run(mtf.mtf_layout(mtf.mtf_mesh_create([("all", 1)]), []), dev, dims)
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("ranks", 2), ("inner", 2)]), rules)
    total = {k: torch.zeros_like(v) for k, v in ref.items()}
    for rank in range(2):
        rec = Recorder(mtf)
        bound = mtf.mtf_layout_bind_ranks(lay, "ranks", 2, rank, rec)
        T, Dm, SL = {}, {}, {}
        for k in list(dev) + list(outs):
            src = dev[k] if k in dev else ref[k]
            T[k], Dm[k], SL[k] = box_of(mtf, bound, src, dims[k])
        O = run(bound, {k: T[k] for k in dev}, Dm)
        ptr_name = {O[k].data_ptr(): k for k in O}
        names = sorted(ptr_name[p] for p, _, _ in rec.started)
        assert names == (["dwk", "dwo", "dwq", "dwv"] if split == "batch" else ["dx", "y"]), names
        for k in O:
            if k in names:
                total[k][SL[k]] += O[k]
            else:
                total[k][SL[k]] = O[k]
    for k in ref:
        close(total[k], ref[k], (split, k))
