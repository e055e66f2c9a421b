"""CPU oracle for the layout-lowered named-dimension einsum and the Transformer blocks built on it.

THIS PACKAGE IS TEST INFRASTRUCTURE.  It is a plain, slow, fp64 restatement of what the paper says
the method computes, used to check the CUDA library.  Only the tests, the smoke check and the
bench's CPU-baseline leg may import it; the product library never does, and the two share no code.

Contents
  einsum_loops.c  the einsum definition as one fp64 loop nest (the only native part)
  named.py        named tensors, dense einsum / reductions / component-wise ops
  mesh.py         mesh, computation layout, legality, per-processor slice boxes
  lowering.py     per-processor simulation: local op on slices, then the group sum (Allreduce)
  blocks.py       feed-forward, attention, layer norm, decoder layer - forward and backward
  stages.py       the same blocks one launch at a time (an einsum plus its fused component-wise stages, or a row reduction)
  cost.py         per-processor cost counts (Table 1, Appendix B)
  chooser.py      exhaustive search for the cheapest legal layout under those counts (Section 11's future work)
  update.py       Algorithm 1 line 3: the parameter update (reading: SGD with momentum and weight decay)
  vocab.py        embedding, logits einsum and softmax cross-entropy over a (split) vocab dimension
  rounding.py     the one rounding step applied where the method stores an intermediate in bf16

Pins (tests that tie each part to something other than itself) are listed in the test files named
test_oracle_*.py.  Parts without an external pin: the bf16 rounding behaviour of the GPU path is
compared by tolerance only ("parity unpinned" beyond the stated tolerances).
"""
from .named import (NT, DenseOps, DuplicateDim, IllegalLayout, NotDivisible, OracleError, SizeMismatch,
                    UnknownDim, einsum_arrays)
from .mesh import Layout, Mesh
from .lowering import LT, LoweredOps
from . import blocks, chooser, cost, rounding, stages, update, vocab

__all__ = ["NT", "DenseOps", "LoweredOps", "LT", "Mesh", "Layout", "blocks", "stages", "cost", "einsum_arrays",
           "OracleError", "DuplicateDim", "UnknownDim", "SizeMismatch", "IllegalLayout", "NotDivisible"]
