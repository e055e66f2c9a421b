"""Pins for the oracle's Transformer blocks (CPU only).

Backward passes are tied to central finite differences of the oracle's own forward pass with a
scalar loss  sum(y * G)  for a fixed random G (a wrong sign, a dropped term or a transposed operand
in any gradient formula fails here).  Forward passes are tied to textbook special cases computed
with numpy (relu(xw+b)v, softmax(QK^T/sqrt(d))V, standardisation) and to invariants (softmax rows
sum to one, gradient rows of the logits sum to zero, causal weights are exactly zero above the
diagonal).  Finally every block must give the same result lowered under several layouts.
"""
import numpy as np
import pytest

from oracle import NT, DenseOps, Layout, LoweredOps, Mesh, blocks
import seeded_inputs as si

D = DenseOps()


def rnd(name, dims, scale=1.0, shift=0.0, seed=21):
    shape = [s for _, s in dims]
    return NT(dims, shift + scale * si.normal_f64(seed, name, int(np.prod(shape))).reshape(shape))


def fd_grad(f, t, eps=1e-6):
    """Central finite differences of scalar f with respect to every element of NT t (in place)."""
    g = np.zeros_like(t.a)
    it = np.nditer(t.a, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = t.a[i]
        t.a[i] = old + eps
        fp = f()
        t.a[i] = old - eps
        fm = f()
        t.a[i] = old
        g[i] = (fp - fm) / (2 * eps)
    return g


# ---- feed-forward --------------------------------------------------------------------------------

def ffn_tensors(b=3, l=2, d=4, f=6):
    x = rnd("x", [("batch", b), ("length", l), ("d_model", d)])
    w = rnd("w", [("d_model", d), ("d_ff", f)], 0.5)
    bias = rnd("bias", [("d_ff", f)], 0.3)
    v = rnd("v", [("d_ff", f), ("d_model", d)], 0.5)
    G = rnd("G", [("batch", b), ("length", l), ("d_model", d)])
    return x, w, bias, v, G


def test_ffn_forward_is_relu_xw_plus_bias_times_v():
    x, w, bias, v, _ = ffn_tensors()
    out = blocks.ffn_forward(D, x, w, bias, v)
    X = x.a.reshape(-1, 4)
    want = np.maximum(X @ w.a + bias.a, 0.0) @ v.a
    np.testing.assert_allclose(out["y"].a.reshape(-1, 4), want, rtol=1e-13, atol=1e-13)
    out2 = blocks.ffn_forward(D, x, w, None, v)
    np.testing.assert_allclose(out2["y"].a.reshape(-1, 4), np.maximum(X @ w.a, 0.0) @ v.a, rtol=1e-13, atol=1e-13)


def test_ffn_backward_matches_finite_differences():
    x, w, bias, v, G = ffn_tensors()
    fwd = blocks.ffn_forward(D, x, w, bias, v)
    assert np.abs(fwd["hp"].a).min() > 1e-4          # away from the relu kink
    g = blocks.ffn_backward(D, x, w, v, fwd["h"], G)
    loss = lambda: float((blocks.ffn_forward(D, x, w, bias, v)["y"].a * G.a).sum())
    for name, t in (("dx", x), ("dw", w), ("dbias", bias), ("dv", v)):
        np.testing.assert_allclose(g[name].a, fd_grad(loss, t), rtol=1e-6, atol=1e-7, err_msg=name)
    # identities: dbias is the column sum of dhp; dw = x^T dhp
    np.testing.assert_allclose(g["dbias"].a, g["dhp"].a.reshape(-1, 6).sum(0), rtol=1e-13)
    np.testing.assert_allclose(g["dw"].a, x.a.reshape(-1, 4).T @ g["dhp"].a.reshape(-1, 6), rtol=1e-12, atol=1e-13)


def test_relu_derivative_at_zero_is_zero():
    h = NT([("batch", 1), ("d_ff", 3)], np.array([[0.0, 1.0, 0.0]]))
    x = NT([("batch", 1), ("d_model", 2)], np.ones((1, 2)))
    w = NT([("d_model", 2), ("d_ff", 3)], np.ones((2, 3)))
    v = NT([("d_ff", 3), ("d_model", 2)], np.ones((3, 2)))
    dy = NT([("batch", 1), ("d_model", 2)], np.ones((1, 2)))
    g = blocks.ffn_backward(D, x, w, v, h, dy)
    assert np.array_equal(g["dhp"].a, np.array([[0.0, 2.0, 0.0]]))


# ---- attention -----------------------------------------------------------------------------------

def att_tensors(b=2, l=3, d=4, h=2, k=2):
    x = rnd("ax", [("batch", b), ("length", l), ("d_model", d)])
    wq = rnd("wq", [("d_model", d), ("heads", h), ("d_k", k)], 0.5)
    wk = rnd("wk", [("d_model", d), ("heads", h), ("d_k", k)], 0.5)
    wv = rnd("wv", [("d_model", d), ("heads", h), ("d_v", k)], 0.5)
    wo = rnd("wo", [("heads", h), ("d_v", k), ("d_model", d)], 0.5)
    G = rnd("aG", [("batch", b), ("length", l), ("d_model", d)])
    return x, wq, wk, wv, wo, G


def np_attention(x, wq, wk, wv, wo, causal):
    B, L, Dm = x.shape
    H, K = wq.shape[1], wq.shape[2]
    y = np.zeros((B, L, Dm))
    for b in range(B):
        for h in range(H):
            Q, Kk, V = x[b] @ wq[:, h, :], x[b] @ wk[:, h, :], x[b] @ wv[:, h, :]
            S = Q @ Kk.T / np.sqrt(K)
            if causal:
                S = np.where(np.triu(np.ones((L, L)), 1) > 0, -np.inf, S)
            P = np.exp(S - S.max(1, keepdims=True))
            P /= P.sum(1, keepdims=True)
            y[b] += (P @ V) @ wo[h]
    return y


@pytest.mark.parametrize("causal", [False, True])
def test_attention_forward_special_case_and_invariants(causal):
    x, wq, wk, wv, wo, _ = att_tensors()
    mask = blocks.causal_mask(3) if causal else None
    out = blocks.attention_forward(D, x, wq, wk, wv, wo, mask)
    np.testing.assert_allclose(out["y"].a, np_attention(x.a, wq.a, wk.a, wv.a, wo.a, causal), rtol=1e-12, atol=1e-13)
    P = out["P"].a                                        # [b, h, l, m]
    np.testing.assert_allclose(P.sum(-1), 1.0, rtol=1e-14)
    if causal:
        assert (P[..., np.triu_indices(3, 1)[0], np.triu_indices(3, 1)[1]] == 0.0).all()


def test_single_head_identity_projections_reduce_to_plain_softmax_attention():
    d = 4
    x = rnd("sx", [("batch", 1), ("length", 5), ("d_model", d)])
    eye = np.eye(d).reshape(d, 1, d)
    wq = NT([("d_model", d), ("heads", 1), ("d_k", d)], eye)
    wv = NT([("d_model", d), ("heads", 1), ("d_v", d)], eye)
    wo = NT([("heads", 1), ("d_v", d), ("d_model", d)], np.eye(d).reshape(1, d, d))
    y = blocks.attention_forward(D, x, wq, wq, wv, wo)["y"].a[0]
    X = x.a[0]
    S = X @ X.T / np.sqrt(d)
    P = np.exp(S - S.max(1, keepdims=True))
    P /= P.sum(1, keepdims=True)
    np.testing.assert_allclose(y, P @ X, rtol=1e-13, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_backward_matches_finite_differences(causal):
    x, wq, wk, wv, wo, G = att_tensors()
    mask = blocks.causal_mask(3) if causal else None
    fwd = blocks.attention_forward(D, x, wq, wk, wv, wo, mask)
    g = blocks.attention_backward(D, x, wq, wk, wv, wo, fwd, G)
    loss = lambda: float((blocks.attention_forward(D, x, wq, wk, wv, wo, mask)["y"].a * G.a).sum())
    for name, t in (("dx", x), ("dwq", wq), ("dwk", wk), ("dwv", wv), ("dwo", wo)):
        np.testing.assert_allclose(g[name].a, fd_grad(loss, t), rtol=1e-6, atol=1e-7, err_msg=name)
    np.testing.assert_allclose(g["dlg"].a.sum(-1), 0.0, atol=1e-13)     # softmax gradient rows sum to 0


# ---- layer norm ------------------------------------------------------------------------------------

def test_layernorm_forward_standardises():
    x = rnd("lx", [("batch", 3), ("length", 2), ("d_model", 8)], 2.0, 0.7)
    one = NT([("d_model", 8)], np.ones(8))
    zero = NT([("d_model", 8)], np.zeros(8))
    eps = 1e-6
    y = blocks.layernorm_forward(D, x, one, zero, eps)["y"].a
    np.testing.assert_allclose(y.mean(-1), 0.0, atol=1e-14)
    var = x.a.var(-1)
    np.testing.assert_allclose(y.var(-1), var / (var + eps), rtol=1e-12)
    gamma, beta = rnd("lg", [("d_model", 8)], 0.1, 1.0), rnd("lb", [("d_model", 8)], 0.1)
    y2 = blocks.layernorm_forward(D, x, gamma, beta, eps)["y"].a
    want = (x.a - x.a.mean(-1, keepdims=True)) / np.sqrt(var[..., None] + eps) * gamma.a + beta.a
    np.testing.assert_allclose(y2, want, rtol=1e-12, atol=1e-13)


def test_layernorm_backward_matches_finite_differences():
    x = rnd("lx", [("batch", 2), ("length", 2), ("d_model", 6)], 2.0, 0.7)
    gamma, beta = rnd("lg", [("d_model", 6)], 0.1, 1.0), rnd("lb", [("d_model", 6)], 0.1)
    G = rnd("lG", x.dims)
    eps = 1e-6
    fwd = blocks.layernorm_forward(D, x, gamma, beta, eps)
    g = blocks.layernorm_backward(D, gamma, fwd, G)
    loss = lambda: float((blocks.layernorm_forward(D, x, gamma, beta, eps)["y"].a * G.a).sum())
    for name, t in (("dx", x), ("dgamma", gamma), ("dbeta", beta)):
        np.testing.assert_allclose(g[name].a, fd_grad(loss, t), rtol=1e-6, atol=1e-7, err_msg=name)


# ---- decoder layer ---------------------------------------------------------------------------------

def layer_params(d=4, h=2, k=2, f=6, zero_sublayers=False):
    p = {"wq": rnd("wq", [("d_model", d), ("heads", h), ("d_k", k)], 0.5),
         "wk": rnd("wk", [("d_model", d), ("heads", h), ("d_k", k)], 0.5),
         "wv": rnd("wv", [("d_model", d), ("heads", h), ("d_v", k)], 0.5),
         "wo": rnd("wo", [("heads", h), ("d_v", k), ("d_model", d)], 0.5),
         "g1": rnd("g1", [("d_model", d)], 0.1, 1.0), "b1": rnd("b1", [("d_model", d)], 0.1),
         "w": rnd("w", [("d_model", d), ("d_ff", f)], 0.5), "bias": rnd("bias", [("d_ff", f)], 0.3),
         "v": rnd("v", [("d_ff", f), ("d_model", d)], 0.5),
         "g2": rnd("g2", [("d_model", d)], 0.1, 1.0), "b2": rnd("b2", [("d_model", d)], 0.1)}
    if zero_sublayers:
        for k_ in ("wo", "v"):
            p[k_] = NT(p[k_].dims, np.zeros_like(p[k_].a))
    return p


def test_decoder_layer_with_zero_sublayers_is_two_layernorms():
    x = rnd("dx", [("batch", 2), ("length", 3), ("d_model", 4)])
    p = layer_params(zero_sublayers=True)
    out = blocks.decoder_layer_forward(D, x, p, blocks.causal_mask(3), 1e-6)["out"].a
    a = blocks.layernorm_forward(D, x, p["g1"], p["b1"], 1e-6)["y"]
    want = blocks.layernorm_forward(D, a, p["g2"], p["b2"], 1e-6)["y"].a
    np.testing.assert_allclose(out, want, rtol=1e-13, atol=1e-14)


def test_decoder_layer_backward_matches_finite_differences():
    x = rnd("dx", [("batch", 2), ("length", 3), ("d_model", 4)])
    p = layer_params()
    mask = blocks.causal_mask(3)
    G = rnd("dG", x.dims)
    fwd = blocks.decoder_layer_forward(D, x, p, mask, 1e-6)
    assert np.abs(fwd["ffn"]["hp"].a).min() > 1e-4
    g = blocks.decoder_layer_backward(D, x, p, fwd, G)
    loss = lambda: float((blocks.decoder_layer_forward(D, x, p, mask, 1e-6)["out"].a * G.a).sum())
    names = {"dx": x, "dwq": p["wq"], "dwk": p["wk"], "dwv": p["wv"], "dwo": p["wo"], "dg1": p["g1"], "db1": p["b1"],
             "dw": p["w"], "dbias": p["bias"], "dv": p["v"], "dg2": p["g2"], "db2": p["b2"]}
    for name, t in names.items():
        np.testing.assert_allclose(g[name].a, fd_grad(loss, t), rtol=2e-6, atol=2e-7, err_msg=name)


# ---- the blocks under layouts: same result as un-split ------------------------------------------------

LAYOUTS = [
    ([("all", 2)], [("batch", "all")]),
    ([("all", 2)], [("d_ff", "all"), ("heads", "all")]),
    ([("rows", 2), ("cols", 2)], [("batch", "rows"), ("d_ff", "cols"), ("heads", "cols")]),
    ([("rows", 2), ("cols", 2)], [("batch", "rows"), ("d_ff", "cols"), ("heads", "cols"), ("vocab", "cols")]),
    ([("all", 2)], []),
]


@pytest.mark.parametrize("mesh_dims,rules", LAYOUTS)
def test_decoder_layer_lowered_equals_dense(mesh_dims, rules):
    x = rnd("dx", [("batch", 2), ("length", 3), ("d_model", 4)])
    p = layer_params()
    mask = blocks.causal_mask(3)
    G = rnd("dG", x.dims)
    fd = blocks.decoder_layer_forward(D, x, p, mask, 1e-6)
    gd = blocks.decoder_layer_backward(D, x, p, fd, G)
    ops = LoweredOps(Layout(Mesh(mesh_dims), rules))
    lp = {k: ops.lower(v) for k, v in p.items()}
    lx = ops.lower(x)
    fl = blocks.decoder_layer_forward(ops, lx, lp, ops.lower(mask), 1e-6)
    gl = blocks.decoder_layer_backward(ops, lx, lp, fl, ops.lower(G))
    np.testing.assert_allclose(ops.to_global(fl["out"]).a, fd["out"].a, rtol=1e-12, atol=1e-13)
    for k in gd:
        np.testing.assert_allclose(ops.to_global(gl[k]).a, gd[k].a, rtol=1e-11, atol=1e-12, err_msg=k)
    tags = [e[0] for e in ops.allreduce_log]
    if rules == [("batch", "all")]:
        # data parallel: only gradient sums over batch are allreduced (Algorithm 1 / Section 8.1)
        assert len(tags) == 12 - 1 and "reduce_max" not in tags     # every parameter gradient; dx none
    if not rules:
        assert tags == []
