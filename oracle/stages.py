"""TEST INFRASTRUCTURE.  The blocks of blocks.py one LAUNCH at a time.

The GPU path stores the result of every einsum (rounded to its storage type) before the next one
reads it.  To hold each launch to the single-einsum tolerance, a test feeds the launch's oracle with
the inputs the GPU launch actually read (downloaded, widened exactly to fp64) and compares the
launch's output.  Every function here is therefore one einsum of Section 6 plus the component-wise
stages that ride in its output (Section 6 "Component-wise Operations", Section 7 broadcasting), or
one row reduction (Section 6 "Reduction"); all arithmetic is fp64 and nothing is rounded.

The tensors may be sub-tensors gathered by the caller (sampled tokens, sampled hidden units, sampled
(batch, head) pairs): the formulas only use dimension names.  Pins: composed in the order of
blocks.py these functions reproduce blocks.py's results, which are themselves pinned by finite
differences and special cases (tests/test_oracle_stages.py).
"""
from __future__ import annotations

import numpy as np

from .named import NT, DenseOps

_ops = DenseOps()


def contraction(a, b, out_names, scale=1.0, bias=None, relu=False, relu_mask=None, residual=None):
    """One einsum with the fused component-wise stages, in the order the boundary defines:
    t = scale * sum(a b);  t += bias (broadcast);  t = max(t, 0) if relu;  t = t where relu_mask > 0 else 0;
    the returned `presum` is t at this point (what a fused reduce_sum adds up);  out = t + residual."""
    t = _ops.einsum([a, b], out_names)
    if scale != 1.0:
        t = _ops.scale(t, scale)
    if bias is not None:
        t = _ops.add(t, bias)
    if relu:
        t = _ops.relu(t)
    if relu_mask is not None:
        t = _ops.mul(t, _ops.positive(relu_mask))
    out = _ops.add(t, residual) if residual is not None else t
    return out, t


def reduce_sum(x, out_names):
    return _ops.reduce_sum(x, out_names)


def softmax_last(lg, causal_query_pos=None):
    """P = exp(lg - max) / sum exp(lg - max) over the LAST dimension.  ``causal_query_pos``: for every
    row (all leading dims, as an integer array of that shape) the query position l; entries with
    memory position m > l are excluded (their weight is exactly 0)."""
    x = lg.a.copy()
    if causal_query_pos is not None:
        m = np.arange(x.shape[-1])
        x = np.where(m > np.asarray(causal_query_pos)[..., None], -np.inf, x)
    e = np.exp(x - x.max(-1, keepdims=True))
    return NT(lg.dims, e / e.sum(-1, keepdims=True))


def softmax_last_backward(P, dP):
    """dlg = P * (dP - sum_last(dP * P))."""
    row = (dP.a * P.a).sum(-1, keepdims=True)
    return NT(P.dims, P.a * (dP.a - row))


def layernorm_rows(x, gamma, beta, eps):
    """Rows of y = gamma * (x - mu) * r + beta with mu, r = (var + eps)^-1/2 over the last dimension
    (biased variance).  Returns y, mu, r."""
    mu = x.a.mean(-1, keepdims=True)
    xc = x.a - mu
    r = 1.0 / np.sqrt((xc * xc).mean(-1, keepdims=True) + eps)
    return NT(x.dims, xc * r * gamma.a + beta.a), mu[..., 0], r[..., 0]


def layernorm_backward_rows(x, dy, gamma, eps, residual=None):
    """Rows of dx = r (g - mean(g) - xh mean(g xh)) (+ residual), g = dy * gamma, xh = (x - mu) r."""
    mu = x.a.mean(-1, keepdims=True)
    xc = x.a - mu
    r = 1.0 / np.sqrt((xc * xc).mean(-1, keepdims=True) + eps)
    xh = xc * r
    g = dy.a * gamma.a
    dx = r * (g - g.mean(-1, keepdims=True) - xh * (g * xh).mean(-1, keepdims=True))
    if residual is not None:
        dx = dx + residual.a
    return NT(x.dims, dx)


def layernorm_param_grads(x, dy, eps, cols=None):
    """dgamma[j] = sum over rows of dy[., j] * xh[., j];  dbeta[j] = sum over rows of dy[., j], for the
    columns ``cols`` (all when None).  x, dy: [rows..., d] with ALL rows (the sums run over them)."""
    x2 = x.a.reshape(-1, x.a.shape[-1])
    dy2 = dy.a.reshape(-1, x.a.shape[-1])
    mu = x2.mean(-1, keepdims=True)
    var = ((x2 - mu) ** 2).mean(-1, keepdims=True)
    r = 1.0 / np.sqrt(var + eps)
    cols = np.arange(x2.shape[1]) if cols is None else np.asarray(cols)
    xh = (x2[:, cols] - mu) * r
    return (dy2[:, cols] * xh).sum(0), dy2[:, cols].sum(0)
