"""Pins of oracle/stages.py (the blocks one launch at a time): composed in the order of the block
functions - which are pinned by finite differences and special cases in test_oracle_blocks.py - the
stage functions must reproduce the blocks' results up to fp64 rounding; the softmax and layer-norm
rows are also held to their defining properties."""
import numpy as np

import seeded_inputs as si
from oracle import NT, DenseOps, blocks, stages

ops = DenseOps()


def close(a, b, tol=1e-11):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    assert a.shape == b.shape
    assert np.max(np.abs(a - b)) <= tol * max(1.0, np.max(np.abs(b)))


def test_ffn_stages_compose_to_the_block():
    B, L, D, F = 3, 5, 8, 12
    x = NT([("batch", B), ("length", L), ("d_model", D)], si.normal(1, "x", [B, L, D], "f32").f64)
    dy = NT(x.dims, si.normal(1, "dy", [B, L, D], "f32").f64)
    w = NT([("d_model", D), ("d_ff", F)], si.normal(1, "w", [D, F], "f32", D ** -0.5).f64)
    v = NT([("d_ff", F), ("d_model", D)], si.normal(1, "v", [F, D], "f32", F ** -0.5).f64)
    bias = NT([("d_ff", F)], si.normal(1, "b", [F], "f32", 0.1).f64)
    f = blocks.ffn_forward(ops, x, w, bias, v)
    g = blocks.ffn_backward(ops, x, w, v, f["h"], dy)
    tok = ["batch", "length"]
    h, _ = stages.contraction(x, w, tok + ["d_ff"], bias=bias, relu=True)
    y, _ = stages.contraction(h, v, tok + ["d_model"])
    dhp, pre = stages.contraction(dy, v, tok + ["d_ff"], relu_mask=h)
    dv, _ = stages.contraction(h, dy, ["d_ff", "d_model"])
    dw, _ = stages.contraction(x, dhp, ["d_model", "d_ff"])
    dx, _ = stages.contraction(dhp, w, tok + ["d_model"], residual=x)
    close(h.a, f["h"].a); close(y.a, f["y"].a); close(dhp.a, g["dhp"].a); close(dv.a, g["dv"].a); close(dw.a, g["dw"].a)
    close(dx.a, g["dx"].a + x.a)
    close(stages.reduce_sum(pre, ["d_ff"]).a, g["dbias"].a)
    # the order of the fused stages: scale first, bias next, relu, mask, residual last
    out, pre = stages.contraction(x, w, tok + ["d_ff"], scale=-2.0, bias=bias, relu=True, relu_mask=f["hp"], residual=f["hp"])
    want_pre = np.maximum(-2.0 * np.einsum("bld,df->blf", x.a, w.a) + bias.a, 0.0) * (f["hp"].a > 0)
    close(pre.a, want_pre); close(out.a, want_pre + f["hp"].a)


def test_attention_stages_compose_to_the_block():
    B, L, D, H, K = 2, 6, 8, 2, 4
    mk = lambda n, shape, s=1.0: si.normal(2, n, shape, "f32", s).f64
    x = NT([("batch", B), ("length", L), ("d_model", D)], mk("x", [B, L, D]))
    dy = NT(x.dims, mk("dy", [B, L, D]))
    wq = NT([("d_model", D), ("heads", H), ("d_k", K)], mk("wq", [D, H, K], D ** -0.5))
    wk = NT(wq.dims, mk("wk", [D, H, K], D ** -0.5))
    wv = NT([("d_model", D), ("heads", H), ("d_v", K)], mk("wv", [D, H, K], D ** -0.5))
    wo = NT([("heads", H), ("d_v", K), ("d_model", D)], mk("wo", [H, K, D], (H * K) ** -0.5))
    s = K ** -0.5
    for causal in (False, True):
        f = blocks.attention_forward(ops, x, wq, wk, wv, wo, blocks.causal_mask(L) if causal else None)
        g = blocks.attention_backward(ops, x, wq, wk, wv, wo, f, dy)
        xm = ops.rename(x, "length", "memory_length")
        q, _ = stages.contraction(x, wq, ["batch", "length", "heads", "d_k"])
        kk, _ = stages.contraction(xm, wk, ["batch", "memory_length", "heads", "d_k"])
        vv, _ = stages.contraction(xm, wv, ["batch", "memory_length", "heads", "d_v"])
        lg, _ = stages.contraction(q, kk, ["batch", "heads", "length", "memory_length"], scale=s)
        pos = np.broadcast_to(np.arange(L), (B, H, L)) if causal else None
        P = stages.softmax_last(lg, pos)
        o, _ = stages.contraction(P, vv, ["batch", "length", "heads", "d_v"])
        y, _ = stages.contraction(o, wo, ["batch", "length", "d_model"])
        for a_, b_ in ((q, f["q"]), (kk, f["kk"]), (vv, f["vv"]), (P, f["P"]), (o, f["o"]), (y, f["y"])):
            close(a_.a, b_.a)
        assert np.allclose(P.a.sum(-1), 1.0)
        if causal:
            iu = np.triu_indices(L, 1)
            assert (P.a[..., iu[0], iu[1]] == 0.0).all()
        dwo, _ = stages.contraction(o, dy, ["heads", "d_v", "d_model"])
        do, _ = stages.contraction(dy, wo, ["batch", "length", "heads", "d_v"])
        dP, _ = stages.contraction(do, vv, ["batch", "heads", "length", "memory_length"])
        dlg = stages.softmax_last_backward(P, dP)
        dvv, _ = stages.contraction(P, do, ["batch", "memory_length", "heads", "d_v"])
        dq, _ = stages.contraction(dlg, kk, ["batch", "length", "heads", "d_k"], scale=s)
        dkk, _ = stages.contraction(dlg, q, ["batch", "memory_length", "heads", "d_k"], scale=s)
        dwq, _ = stages.contraction(x, dq, ["d_model", "heads", "d_k"])
        dwk, _ = stages.contraction(xm, dkk, ["d_model", "heads", "d_k"])
        dwv, _ = stages.contraction(xm, dvv, ["d_model", "heads", "d_v"])
        t1, _ = stages.contraction(dq, wq, ["batch", "length", "d_model"])
        t2, _ = stages.contraction(dkk, wk, ["batch", "memory_length", "d_model"])
        t3, _ = stages.contraction(dvv, wv, ["batch", "memory_length", "d_model"])
        for a_, k_ in ((dwo, "dwo"), (do, "do"), (dlg, "dlg"), (dvv, "dvv"), (dq, "dq"), (dkk, "dkk"), (dwq, "dwq"), (dwk, "dwk"), (dwv, "dwv")):
            close(a_.a, g[k_].a)
        close(t1.a + t2.a + t3.a, g["dx"].a)
        assert np.allclose(dlg.a.sum(-1), 0.0, atol=1e-12)


def test_layernorm_stages_match_the_block_and_its_definition():
    R, D, eps = 7, 16, 1e-6
    x = NT([("tok", R), ("d_model", D)], si.normal(3, "x", [R, D], "f32", 2.0, 0.5).f64)
    dy = NT(x.dims, si.normal(3, "dy", [R, D], "f32").f64)
    res = NT(x.dims, si.normal(3, "res", [R, D], "f32").f64)
    gamma = NT([("d_model", D)], si.normal(3, "g", [D], "f32", 0.1, 1.0).f64)
    beta = NT([("d_model", D)], si.normal(3, "b", [D], "f32", 0.1).f64)
    f = blocks.layernorm_forward(ops, x, gamma, beta, eps)
    g = blocks.layernorm_backward(ops, gamma, f, dy)
    y, mu, r = stages.layernorm_rows(x, gamma, beta, eps)
    close(y.a, f["y"].a)
    close(mu, x.a.mean(-1)); close(r, 1.0 / np.sqrt(x.a.var(-1) + eps))
    close(stages.layernorm_backward_rows(x, dy, gamma, eps).a, g["dx"].a)
    close(stages.layernorm_backward_rows(x, dy, gamma, eps, res).a, g["dx"].a + res.a)
    dg, db = stages.layernorm_param_grads(x, dy, eps)
    close(dg, g["dgamma"].a); close(db, g["dbeta"].a)
    cols = [0, 5, D - 1]
    dg2, db2 = stages.layernorm_param_grads(x, dy, eps, cols)
    close(dg2, g["dgamma"].a[cols]); close(db2, g["dbeta"].a[cols])
    # rows are independent: a subset of rows gives the same rows
    sub = NT([("tok", 3), ("d_model", D)], x.a[[1, 4, 6]])
    close(stages.layernorm_rows(sub, gamma, beta, eps)[0].a, f["y"].a[[1, 4, 6]])
