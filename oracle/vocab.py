"""TEST INFRASTRUCTURE.  The `vocab` dimension of the Transformer layout (Section 9: vocab, d_ff and
heads are the split dimensions; every expensive operation has exactly one of them): token embedding,
the logits einsum and the softmax cross-entropy loss, forward and backward, written with the
operations of Section 6 so that they run un-split (DenseOps) or slice by slice (LoweredOps):

  embedding      x[t, d]   = sum_v onehot(ids)[t, v] E[v, d]           an einsum that reduces `vocab`
  logits         lg[t, v]  = sum_d h[t, d] Wout[d, v]
  loss           mx[t] = max_v lg;  se[t] = sum_v exp(lg - mx);  lse = mx + log se      ("Reduction":
                 picked[t] = sum_v lg * onehot(target);  loss[t] = lse - picked          local + group)
  backward       dlg[t, v] = (exp(lg - lse) - onehot(target)) * dloss[t]
                 dh[t, d]  = sum_v dlg Wout[d, v]   (reduces vocab);   dWout[d, v] = sum_t h dlg
                 dE[v, d]  = sum_t onehot(ids)[t, v] dx[t, d]          (reduces the token dimensions)
The Transformer's loss is not spelled out in the paper; this is the usual maximum-likelihood loss of
the model it refers to (Vaswani et al.), per token, un-smoothed.
"""
from __future__ import annotations

import numpy as np

from .named import NT


def one_hot(ids, tok_dims, vocab_dim):
    """ids: integer array shaped like tok_dims -> NT [*tok_dims, vocab] of 0.0 / 1.0."""
    ids = np.asarray(ids)
    V = int(vocab_dim[1])
    a = (ids[..., None] == np.arange(V)).astype(np.float64)
    return NT(list(tok_dims) + [vocab_dim], a)


def embedding_forward(ops, onehot, E):
    tok = list(onehot.names[:-1])
    return ops.einsum([onehot, E], tok + [E.names[1]])


def embedding_backward(ops, onehot, dx, E_names):
    return ops.einsum([onehot, dx], list(E_names))


def xent_forward(ops, h, wout, onehot_target):
    tok = list(h.names[:-1])
    vocab = wout.names[1]
    lg = ops.einsum([h, wout], tok + [vocab])
    mx = ops.reduce_max(lg, tok)
    se = ops.reduce_sum(ops.exp(ops.sub(lg, mx)), tok)
    lse = ops.add(mx, ops.unary(se, np.log))
    picked = ops.reduce_sum(ops.mul(lg, onehot_target), tok)
    return {"logits": lg, "lse": lse, "loss": ops.sub(lse, picked)}


def xent_backward(ops, h, wout, lg, lse, onehot_target, dloss):
    tok = list(h.names[:-1])
    P = ops.exp(ops.sub(lg, lse))
    dlg = ops.mul(ops.sub(P, onehot_target), dloss)
    dh = ops.einsum([dlg, wout], tok + [h.names[-1]])
    dwout = ops.einsum([h, dlg], list(wout.names))
    return {"dlogits": dlg, "dh": dh, "dwout": dwout}
