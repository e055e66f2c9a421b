"""TEST INFRASTRUCTURE.  The Transformer blocks written as named-dim einsums, reductions and
component-wise operations, forward and backward.  Every function takes an ``ops`` object: with
``DenseOps`` it is the un-split mathematics, with ``LoweredOps`` the same sequence is executed slice
by slice with the group sums of Section 6.

Feed-forward block: Section 8, y = Relu(x w + bias) v, and its code fragment (two einsums, a
broadcast add and a relu).  The backward pass is the chain rule written with the same operations;
Section 8.1 notes that the parameter gradients are einsums that reduce out `batch`, Section 8.2 that
the gradient on x reduces out `hidden`.

Attention, layer normalisation and the decoder layer are not spelled out in the paper (Section 9
refers to the Transformer of Vaswani et al.); the formulas used are stated in each docstring.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------------------------------
# Feed-forward block (Section 8)
# --------------------------------------------------------------------------------------------------

def _identity(t):
    return t


def ffn_forward(ops, x, w, bias, v, store=_identity):
    """hp = x.w (+ bias);  h = relu(hp);  y = h.v.
    x: [*tokens, io]   w: [io, hidden]   bias: [hidden] or None   v: [hidden, io].
    ``store`` is applied where a result is kept between two einsums (h): identity = exact
    mathematics, a rounding function = the storage precision of that tensor."""
    tok = list(x.names[:-1])
    hidden = w.names[1]
    hp = ops.einsum([x, w], tok + [hidden])
    if bias is not None:
        hp = ops.add(hp, bias)
    h = store(ops.relu(hp))
    y = ops.einsum([h, v], tok + [v.names[1]])
    return {"hp": hp, "h": h, "y": y}


def ffn_backward(ops, x, w, v, h, dy, store=_identity):
    """dh = dy.v^T;  dhp = dh * [h > 0]  (relu'(0) = 0; h > 0 exactly where hp > 0);
    dv = h^T.dy and dw = x^T.dhp (reduce the token dims);  dbias = sum over tokens of dhp;
    dx = dhp.w^T (reduces hidden)."""
    tok = list(x.names[:-1])
    hidden = w.names[1]
    dh = ops.einsum([dy, v], tok + [hidden])
    dhp_exact = ops.mul(dh, ops.positive(h))
    dhp = store(dhp_exact)                       # kept between einsums
    dv = ops.einsum([h, dy], list(v.names))
    dw = ops.einsum([x, dhp], list(w.names))
    dbias = ops.reduce_sum(dhp_exact, [hidden])    # summed before the value is stored
    dx = ops.einsum([dhp, w], list(x.names))
    return {"dhp": dhp, "dv": dv, "dw": dw, "dbias": dbias, "dx": dx}


# --------------------------------------------------------------------------------------------------
# Multi-head attention (reading: Vaswani et al., no projection biases, no dropout)
# --------------------------------------------------------------------------------------------------

def causal_mask(length, memory_length="memory_length", length_name="length"):
    """Additive mask [length, memory_length]: 0 where m <= l, -inf where m > l."""
    from .named import NT
    L = int(length)
    m = np.where(np.arange(L)[None, :] > np.arange(L)[:, None], -np.inf, 0.0)
    return NT([(length_name, L), (memory_length, L)], m)


def attention_forward(ops, x, wq, wk, wv, wo, mask=None, store=_identity, residual=None):
    """x: [batch, length, d_model]; wq, wk: [d_model, heads, d_k]; wv: [d_model, heads, d_v];
    wo: [heads, d_v, d_model].  xm is x with `length` renamed `memory_length` (same data; a tensor
    cannot carry one name twice).
        q[b,l,h,k] = sum_d x wq      kk[b,m,h,k] = sum_d xm wk      vv[b,m,h,v] = sum_d xm wv
        lg[b,h,l,m] = d_k^-1/2 sum_k q kk  (+ mask[l,m])
        P = exp(lg - max_m lg) / sum_m exp(lg - max_m lg)
        o[b,l,h,v] = sum_m P vv      y[b,l,d] = sum_{h,v} o wo  (+ residual)
    ``store`` is applied to q, kk, vv, P and o (kept between einsums); the logits are not stored
    in a narrow type."""
    b, l, d = x.names
    _, h, k = wq.names
    vdim = wv.names[2]
    m = "memory_length"
    s = 1.0 / np.sqrt(float(dict(wq.dims)[k]))
    xm = ops.rename(x, l, m)
    q = store(ops.einsum([x, wq], [b, l, h, k]))
    kk = store(ops.einsum([xm, wk], [b, m, h, k]))
    vv = store(ops.einsum([xm, wv], [b, m, h, vdim]))
    lg = ops.scale(ops.einsum([q, kk], [b, h, l, m]), s)
    if mask is not None:
        lg = ops.add(lg, mask)
    mx = ops.reduce_max(lg, [b, h, l])
    e = ops.exp(ops.sub(lg, mx))
    z = ops.reduce_sum(e, [b, h, l])
    P = store(ops.mul(e, ops.unary(z, lambda a: 1.0 / a)))
    o = store(ops.einsum([P, vv], [b, l, h, vdim]))
    y = ops.einsum([o, wo], [b, l, d])
    if residual is not None:
        y = ops.add(y, residual)
    return {"q": q, "kk": kk, "vv": vv, "P": P, "o": o, "y": y}


def attention_backward(ops, x, wq, wk, wv, wo, saved, dy, store=_identity):
    """dwo[h,v,d] = sum_{b,l} o dy;  do = sum_d dy wo;  dP = sum_v do vv;  dvv = sum_l P do;
    dlg = P * (dP - sum_m dP*P);  dq = s sum_m dlg kk;  dkk = s sum_l dlg q;
    dwq = sum_{b,l} x dq;  dwk = sum_{b,m} xm dkk;  dwv = sum_{b,m} xm dvv;
    dx = sum_{h,k} dq wq + rename_{m->l}(sum_{h,k} dkk wk + sum_{h,v} dvv wv)."""
    b, l, d = x.names
    _, h, k = wq.names
    vdim = wv.names[2]
    m = "memory_length"
    s = 1.0 / np.sqrt(float(dict(wq.dims)[k]))
    q, kk, vv, P, o = saved["q"], saved["kk"], saved["vv"], saved["P"], saved["o"]
    xm = ops.rename(x, l, m)
    dwo = ops.einsum([o, dy], list(wo.names))
    do = store(ops.einsum([dy, wo], [b, l, h, vdim]))
    dP = ops.einsum([do, vv], [b, h, l, m])
    dvv = store(ops.einsum([P, do], [b, m, h, vdim]))
    row = ops.reduce_sum(ops.mul(dP, P), [b, h, l])
    dlg = store(ops.mul(P, ops.sub(dP, row)))
    dq = store(ops.scale(ops.einsum([dlg, kk], [b, l, h, k]), s))
    dkk = store(ops.scale(ops.einsum([dlg, q], [b, m, h, k]), s))
    dwq = ops.einsum([x, dq], list(wq.names))
    dwk = ops.einsum([xm, dkk], list(wk.names))
    dwv = ops.einsum([xm, dvv], list(wv.names))
    dx_q = ops.einsum([dq, wq], [b, l, d])
    dx_m = ops.add(ops.einsum([dkk, wk], [b, m, d]), ops.einsum([dvv, wv], [b, m, d]))
    dx = ops.add(dx_q, ops.rename(dx_m, m, l))
    return {"dwo": dwo, "dwq": dwq, "dwk": dwk, "dwv": dwv, "dx": dx,
            "dq": dq, "dkk": dkk, "dvv": dvv, "dlg": dlg, "do": do}


# --------------------------------------------------------------------------------------------------
# Layer normalisation over the last dimension (reading: biased variance, eps inside the root)
# --------------------------------------------------------------------------------------------------

def layernorm_forward(ops, x, gamma, beta, eps):
    """mu = mean_d x;  var = mean_d (x-mu)^2;  r = (var+eps)^-1/2;  xh = (x-mu) r;  y = gamma*xh + beta."""
    tok = list(x.names[:-1])
    D = float(x.dims[-1][1])
    mu = ops.scale(ops.reduce_sum(x, tok), 1.0 / D)
    xc = ops.sub(x, mu)
    var = ops.scale(ops.reduce_sum(ops.mul(xc, xc), tok), 1.0 / D)
    r = ops.rsqrt_plus(var, eps)
    xh = ops.mul(xc, r)
    y = ops.add(ops.mul(xh, gamma), beta)
    return {"xh": xh, "r": r, "y": y}


def layernorm_backward(ops, gamma, saved, dy):
    """g = dy*gamma;  dx = r (g - mean_d g - xh mean_d(g*xh));  dgamma = sum_tokens dy*xh;  dbeta = sum_tokens dy."""
    xh, r = saved["xh"], saved["r"]
    tok = list(xh.names[:-1])
    dname = xh.names[-1]
    D = float(xh.dims[-1][1])
    g = ops.mul(dy, gamma)
    m1 = ops.scale(ops.reduce_sum(g, tok), 1.0 / D)
    m2 = ops.scale(ops.reduce_sum(ops.mul(g, xh), tok), 1.0 / D)
    dx = ops.mul(ops.sub(ops.sub(g, m1), ops.mul(xh, m2)), r)
    dgamma = ops.reduce_sum(ops.mul(dy, xh), [dname])
    dbeta = ops.reduce_sum(dy, [dname])
    return {"dx": dx, "dgamma": dgamma, "dbeta": dbeta}


# --------------------------------------------------------------------------------------------------
# Decoder layer (reading: post-layer-norm residual blocks, a = LN1(x + Att(x)); out = LN2(a + FFN(a)))
# --------------------------------------------------------------------------------------------------

def decoder_layer_forward(ops, x, p, mask, eps, store=_identity):
    """p: dict with wq, wk, wv, wo, g1, b1, w, bias, v, g2, b2 (already in ops' representation).
    ``store`` additionally applies to the two residual sums s1, s2 and to a (kept for backward)."""
    att = attention_forward(ops, x, p["wq"], p["wk"], p["wv"], p["wo"], mask, store)
    s1 = store(ops.add(x, att["y"]))
    ln1 = layernorm_forward(ops, s1, p["g1"], p["b1"], eps)
    a = store(ln1["y"])
    ffn = ffn_forward(ops, a, p["w"], p["bias"], p["v"], store)
    s2 = store(ops.add(a, ffn["y"]))
    ln2 = layernorm_forward(ops, s2, p["g2"], p["b2"], eps)
    return {"att": att, "ln1": ln1, "a": a, "ffn": ffn, "ln2": ln2, "out": ln2["y"]}


def decoder_layer_backward(ops, x, p, saved, dout, store=_identity):
    """Chain rule through the two residual sums (the gradient streams ds2, da, ds1 are stored)."""
    l2 = layernorm_backward(ops, p["g2"], saved["ln2"], dout)
    ds2 = store(l2["dx"])                             # gradient on (a + FFN(a))
    fb = ffn_backward(ops, saved["a"], p["w"], p["v"], saved["ffn"]["h"], ds2, store)
    da = store(ops.add(ds2, fb["dx"]))
    l1 = layernorm_backward(ops, p["g1"], saved["ln1"], da)
    ds1 = store(l1["dx"])                             # gradient on (x + Att(x))
    ab = attention_backward(ops, x, p["wq"], p["wk"], p["wv"], p["wo"], saved["att"], ds1, store)
    dx = ops.add(ds1, ab["dx"])
    return {"dx": dx, "dg2": l2["dgamma"], "db2": l2["dbeta"], "dg1": l1["dgamma"], "db1": l1["dbeta"],
            "dw": fb["dw"], "dbias": fb["dbias"], "dv": fb["dv"],
            "dwq": ab["dwq"], "dwk": ab["dwk"], "dwv": ab["dwv"], "dwo": ab["dwo"]}
