"""The blocks can be captured into a CUDA graph and replayed: no entry point allocates, synchronises or
keeps host state that a replay would miss.  In particular the launches that draw their tiles from a
counter (the independent launches inside the backward passes) leave their counter cleared, so the
second and third replay give bit for bit what the eager calls give."""
import pytest

import seeded_inputs as si
from helpers import to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


def test_ffn_forward_backward_replays_from_a_graph(mtf):
    import torch
    B, L, D, F = 8, 256, 1024, 4096      # 2048 tokens: several waves of tiles in dhp, few tiles in dv / dw / dx
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 8)]), [("d_ff", "all")])
    bf = torch.bfloat16
    t = {"x": to_torch(si.normal(3, "x", [B, L, D], "bf16")), "dy": to_torch(si.normal(3, "dy", [B, L, D], "bf16")),
         "w": to_torch(si.normal(3, "w", [D, F], "bf16", D ** -0.5)), "v": to_torch(si.normal(3, "v", [F, D], "bf16", F ** -0.5)),
         "bias": to_torch(si.normal(3, "bias", [F], "f32", 0.1))}
    h = torch.empty(B, L, F, dtype=bf, device="cuda"); y = torch.empty(B, L, D, dtype=bf, device="cuda"); dx = torch.empty_like(y)
    dw = torch.empty(D, F, device="cuda"); dv = torch.empty(F, D, device="cuda"); dbias = torch.empty(F, device="cuda")
    act, wn, vn, hn = ["batch", "length", "d_model"], ["d_model", "d_ff"], ["d_ff", "d_model"], ["batch", "length", "d_ff"]
    N = {"x": mtf.named(t["x"], act), "dy": mtf.named(t["dy"], act), "w": mtf.named(t["w"], wn), "v": mtf.named(t["v"], vn),
         "bias": mtf.named(t["bias"], ["d_ff"]), "h": mtf.named(h, hn), "y": mtf.named(y, act), "dx": mtf.named(dx, act),
         "dw": mtf.named(dw, wn), "dv": mtf.named(dv, vn), "dbias": mtf.named(dbias, ["d_ff"])}
    ws = torch.empty(mtf.mtf_ffn_workspace_bytes(lay, N["x"], N["w"]), dtype=torch.uint8, device="cuda")
    outs = (h, y, dx, dw, dv, dbias)

    def step():
        mtf.mtf_ffn_forward(lay, N["x"], N["w"], N["bias"], N["v"], N["h"], N["y"], ws)
        mtf.mtf_ffn_backward(lay, N["x"], N["w"], N["v"], N["h"], N["dy"], N["dx"], N["dw"], N["dbias"], N["dv"], ws)

    step()                                   # eager: plans, attributes and lookups happen here
    mtf.mtf_device_status()
    want = [o.clone() for o in outs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for rep in range(3):
        for o in outs:
            o.zero_()
        graph.replay()
        mtf.mtf_device_status()
        for name, o, w_ in zip(("h", "y", "dx", "dw", "dv", "dbias"), outs, want):
            assert torch.equal(o, w_), (rep, name)
    step()                                   # and eager calls still work after the replays
    mtf.mtf_device_status()
    for o, w_ in zip(outs, want):
        assert torch.equal(o, w_)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_forward_backward_replays_from_a_graph(mtf, causal):
    """Both one-launch attention cores, the grouped and multi-term projections and the two independent launches of the
    backward pass (dWo behind the core, dx behind the weight gradients) inside one captured graph."""
    import torch
    B, L, D, H, K = 12, 256, 512, 8, 64      # 96 (batch, head) pairs: blocks with one and with no pair in the core's grid
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("rows", 4), ("cols", 4)]), [("batch", "rows"), ("heads", "cols")])
    dims = {"x": [("batch", B), ("length", L), ("d_model", D)], "wq": [("d_model", D), ("heads", H), ("d_k", K)],
            "wk": [("d_model", D), ("heads", H), ("d_k", K)], "wv": [("d_model", D), ("heads", H), ("d_v", K)],
            "wo": [("heads", H), ("d_v", K), ("d_model", D)], "dy": [("batch", B), ("length", L), ("d_model", D)]}
    scale = {"x": 1.0, "dy": 1.0, "wq": D ** -0.5, "wk": D ** -0.5, "wv": D ** -0.5, "wo": (H * K) ** -0.5}
    dev = {k: to_torch(si.normal(21, k, [s for _, s in d], "bf16", scale[k])) for k, d in dims.items()}
    N = {k: mtf.named(dev[k], [n for n, _ in d]) for k, d in dims.items()}
    nm = mtf.named
    E = lambda *s: torch.empty(*s, device="cuda", dtype=torch.bfloat16)
    F = lambda *s: torch.empty(*s, device="cuda", dtype=torch.float32)
    q, kk, vv, o = E(B, L, H, K), E(B, L, H, K), E(B, L, H, K), E(B, L, H, K)
    P, y, dx = E(B, H, L, L), E(B, L, D), E(B, L, D)
    dwq, dwk, dwv, dwo = F(D, H, K), F(D, H, K), F(D, H, K), F(H, K, D)
    ws = torch.empty(mtf.mtf_attention_workspace_bytes(lay, N["x"], N["wq"], N["wv"]), dtype=torch.uint8, device="cuda")
    Q = nm(q, ["batch", "length", "heads", "d_k"]); KK = nm(kk, ["batch", "memory_length", "heads", "d_k"])
    VV = nm(vv, ["batch", "memory_length", "heads", "d_v"]); PP = nm(P, ["batch", "heads", "length", "memory_length"])
    O = nm(o, ["batch", "length", "heads", "d_v"]); Y = nm(y, ["batch", "length", "d_model"])
    outs = (q, kk, vv, o, P, y, dx, dwq, dwk, dwv, dwo)

    def step():
        mtf.mtf_attention_forward(lay, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], causal, None, Q, KK, VV, PP, O, Y, ws)
        mtf.mtf_attention_backward(lay, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], Q, KK, VV, PP, O, N["dy"], None, nm(dx, ["batch", "length", "d_model"]),
                                   nm(dwq, ["d_model", "heads", "d_k"]), nm(dwk, ["d_model", "heads", "d_k"]), nm(dwv, ["d_model", "heads", "d_v"]),
                                   nm(dwo, ["heads", "d_v", "d_model"]), ws, causal=causal)

    step()
    mtf.mtf_device_status()
    want = [t.clone() for t in outs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for rep in range(3):
        for t in outs:
            t.zero_()
        graph.replay()
        mtf.mtf_device_status()
        for i, (t, w_) in enumerate(zip(outs, want)):
            assert torch.equal(t, w_), (rep, i)
