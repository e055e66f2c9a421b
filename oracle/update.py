"""TEST INFRASTRUCTURE.  The parameter update of Algorithm 1, line 3: W(t+1) = Update(W(t), gradient).

The paper leaves `Update` open.  Reading taken (stated in the design notes): stochastic gradient
descent with optional momentum and decoupled weight decay on an fp32 master copy, plus the bf16
working copy the contractions read:
    m  <- momentum * m + g                      (m omitted when momentum = 0: m = g)
    W  <- W - lr * (m + weight_decay * W)
    Wb <- round_to_nearest_even_bf16(W)
Every processor updates its own slice of every parameter (Algorithm 1: "each processor updates its
own copy"); the update is component-wise (Section 6), so it is local under every layout and the
slices of the result are the slices of the dense result.
"""
from __future__ import annotations

import numpy as np


def sgd_update(master, grad, mom, lr, momentum=0.0, weight_decay=0.0):
    """fp64 arrays in, fp64 arrays out: (new master, new momentum or None)."""
    master = np.asarray(master, dtype=np.float64)
    g = np.asarray(grad, dtype=np.float64)
    if mom is not None:
        m = momentum * np.asarray(mom, dtype=np.float64) + g
    else:
        m = g
    new = master - lr * (m + weight_decay * master)
    return new, (m if mom is not None else None)


def lowered_update(ops, master, grad, mom, lr, momentum=0.0, weight_decay=0.0):
    """The same update written with the component-wise operations of ``ops`` (DenseOps or LoweredOps):
    every processor works on its slices only."""
    m = ops.add(ops.scale(mom, momentum), grad) if mom is not None else grad
    step = ops.add(m, ops.scale(master, weight_decay))
    return ops.sub(master, ops.scale(step, lr)), (m if mom is not None else None)
