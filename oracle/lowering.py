"""TEST INFRASTRUCTURE.  The lowered ("SPMD") computation, simulated processor by processor.

Section 4: each tensor is represented by one slice per processor; each operation is one local
operation per processor, some followed by a collective.  Section 6:
  * component-wise ops are purely local;
  * a reduction is a local reduction followed by an Allreduce across the mesh dimensions of the
    reduced-out split tensor dimensions;
  * an einsum is a local einsum of the processor's input slices followed by an Allreduce across the
    mesh dimensions of the reduced-out split tensor dimensions.
The Allreduce within a group (all processors that agree on the remaining mesh dimensions; Section 8
calls the 2-D case a partitioned Allreduce) leaves every member with the sum, taken here in
ascending processor order.  Every processor is simulated, replicas included.
"""
from __future__ import annotations

import numpy as np

from .mesh import Layout
from .named import (NT, DenseOps, OracleError, SizeMismatch, UnknownDim, einsum_arrays,
                    resolve_out_dims, union_dims)


class LT:
    """A lowered tensor: global ``dims`` plus one fp64 slice per processor."""

    __slots__ = ("dims", "slices")

    def __init__(self, dims, slices):
        self.dims = tuple(dims)
        self.slices = list(slices)

    @property
    def names(self):
        return tuple(n for n, _ in self.dims)


class LoweredOps:
    """Same interface as ``DenseOps`` but acting on per-processor slices under a layout."""

    def __init__(self, layout: Layout):
        self.layout = layout
        self.mesh = layout.mesh
        self._dense = DenseOps()
        self.allreduce_log = []   # (op, reduced mesh-dim indices, values per processor)

    # -- moving between the global and the lowered representation -----------------------------------
    def lower(self, x: NT) -> LT:
        return LT(x.dims, [self.layout.slice_of(x.dims, x.a, p) for p in range(self.mesh.P)])

    def to_global(self, x: LT) -> NT:
        """Assemble the global tensor from the slices and check the paper's consistency statement:
        processors whose slices cover the same box hold identical values (bitwise)."""
        out = np.full([s for _, s in x.dims], np.nan, dtype=np.float64)
        written = {}
        for p in range(self.mesh.P):
            offs, sizes = self.layout.slice_box(x.dims, p)
            key = tuple(offs)
            if key in written:
                if not np.array_equal(x.slices[written[key]], x.slices[p]):
                    raise AssertionError(f"replicas on processors {written[key]} and {p} differ")
                continue
            written[key] = p
            out[tuple(slice(o, o + t) for o, t in zip(offs, sizes))] = x.slices[p]
        if np.isnan(out).any():
            raise AssertionError("slices do not cover the tensor")
        return NT(x.dims, out)

    # -- the group sum ("Allreduce") ---------------------------------------------------------------
    def _allreduce(self, partials, over, fn=np.add, tag="einsum"):
        if not over:
            return partials
        out = []
        for p in range(self.mesh.P):
            g = self.mesh.group(p, over)
            acc = partials[g[0]].copy()
            for q in g[1:]:
                acc = fn(acc, partials[q])
            out.append(acc)
        self.allreduce_log.append((tag, tuple(sorted(over)), int(partials[0].size)))
        return out

    def _reduced_mesh_dims(self, in_dim_lists, out_dims):
        out_names = [n for n, _ in out_dims]
        over = set()
        for n, _ in union_dims(in_dim_lists):
            if n not in out_names:
                j = self.layout.mesh_dim_of(n)
                if j is not None:
                    over.add(j)
        return over

    # -- einsum -------------------------------------------------------------------------------------
    def einsum(self, inputs, out_names):
        in_dims = [t.dims for t in inputs]
        out_dims = resolve_out_dims(in_dims, out_names)
        self.layout.check_iteration_space(in_dims + [out_dims])
        for d in in_dims + [out_dims]:
            self.layout.tensor_layout(d)
        partials = []
        for p in range(self.mesh.P):
            loc_in = [self.layout.slice_dims(t.dims, p) for t in inputs]
            loc_out = self.layout.slice_dims(out_dims, p)
            partials.append(einsum_arrays(loc_in, [t.slices[p] for t in inputs], loc_out))
        over = self._reduced_mesh_dims(in_dims, out_dims)
        return LT(out_dims, self._allreduce(partials, over))

    # -- component-wise -----------------------------------------------------------------------------
    def _binary(self, x, y, name):
        big, small = (y, x) if len(y.dims) > len(x.dims) else (x, y)
        for n, s in small.dims:
            if n not in big.names:
                raise UnknownDim(n)
            if dict(big.dims)[n] != s:
                raise SizeMismatch(n)
        out = []
        for p in range(self.mesh.P):
            a = NT(self.layout.slice_dims(x.dims, p), x.slices[p])
            b = NT(self.layout.slice_dims(y.dims, p), y.slices[p])
            out.append(getattr(self._dense, name)(a, b).a)
        return LT(big.dims, out)

    def add(self, x, y):
        return self._binary(x, y, "add")

    def sub(self, x, y):
        return self._binary(x, y, "sub")

    def mul(self, x, y):
        return self._binary(x, y, "mul")

    def unary(self, x, fn):
        return LT(x.dims, [fn(s) for s in x.slices])

    def relu(self, x):
        return self.unary(x, lambda a: np.maximum(a, 0.0))

    def positive(self, x):
        return self.unary(x, lambda a: (a > 0.0).astype(np.float64))

    def exp(self, x):
        return self.unary(x, np.exp)

    def scale(self, x, c):
        return self.unary(x, lambda a: a * float(c))

    def rsqrt_plus(self, x, eps):
        return self.unary(x, lambda a: 1.0 / np.sqrt(a + eps))

    # -- reductions ---------------------------------------------------------------------------------
    def _reduce(self, x, out_names, name, fn):
        out_dims = resolve_out_dims([x.dims], out_names)
        partials = []
        for p in range(self.mesh.P):
            loc = NT(self.layout.slice_dims(x.dims, p), x.slices[p])
            partials.append(getattr(self._dense, name)(loc, [n for n, _ in out_dims]).a)
        over = self._reduced_mesh_dims([x.dims], out_dims)
        return LT(out_dims, self._allreduce(partials, over, fn, tag=name))

    def reduce_sum(self, x, out_names):
        return self._reduce(x, out_names, "reduce_sum", np.add)

    def reduce_max(self, x, out_names):
        return self._reduce(x, out_names, "reduce_max", np.maximum)

    def rename(self, x, old, new):
        """Rename one dimension: the reshape of Section 6.1 with one name changed."""
        return self.reshape(x, [new if n == old else n for n in x.names])

    def reshape(self, x, out_names):
        """Reshape that keeps the sizes and changes dimension names (Section 6.1), hence possibly the
        layout.  Per mesh dimension the paper names three patterns:
          * a tensor dimension split over it in the input but none in the output: Allgather over that
            mesh dimension (every member of the group ends with the concatenation, in coordinate order);
          * none in the input, one in the output: no communication, each processor keeps its stripe;
          * different tensor dimensions in input and output: Alltoall over that mesh dimension (here
            carried out as its definition: gather the group's blocks, keep the own stripe of the other
            dimension; the elements a processor receives are counted as an Alltoall's).
        All gathers run before all slicing, so that every step acts on whole stripes.
        ``reshape_log`` receives (mesh-dim index, pattern, elements received per processor)."""
        in_dims = x.dims
        if len(out_names) != len(in_dims):
            raise SizeMismatch("reshape keeps the number and the sizes of the dimensions")
        out_dims = tuple((n, s) for n, (_, s) in zip(out_names, in_dims))
        tl_in = {j: i for i, j in self.layout.tensor_layout(in_dims).items()}        # mesh dim -> position
        tl_out = {j: i for i, j in self.layout.tensor_layout(out_dims).items()}
        slices = [s.copy() for s in x.slices]
        self.reshape_log = getattr(self, "reshape_log", [])
        changed = [j for j in range(len(self.mesh.shape)) if tl_in.get(j) != tl_out.get(j)]
        for j in changed:                                   # gathers
            if j not in tl_in:
                continue
            pos, m = tl_in[j], self.mesh.shape[j]
            local = int(slices[0].size)
            gathered = []
            for p in range(self.mesh.P):
                grp = self.mesh.group(p, {j})               # ascending processor order = ascending coordinate j
                gathered.append(np.concatenate([slices[q] for q in grp], axis=pos))
            slices = gathered
            if j in tl_out:                                 # an Alltoall keeps 1/m of what the gather brought
                self.reshape_log.append((j, "alltoall", local * (m - 1) // m))
            else:
                self.reshape_log.append((j, "allgather", local * (m - 1)))
        for j in changed:                                   # local slicing
            if j not in tl_out:
                continue
            pos, m = tl_out[j], self.mesh.shape[j]
            kept = []
            for p in range(self.mesh.P):
                c = self.mesh.coords(p)[j]
                t = slices[p].shape[pos] // m
                idx = [slice(None)] * slices[p].ndim
                idx[pos] = slice(c * t, (c + 1) * t)
                kept.append(np.require(slices[p][tuple(idx)], requirements="C").copy())
            slices = kept
            if j not in tl_in:
                self.reshape_log.append((j, "slice", 0))
        return LT(out_dims, slices)

    def transpose(self, x, out_names):
        """Same dimensions in another storage order: purely local (the layout goes by names)."""
        perm = [x.names.index(n) for n in out_names]
        return LT([x.dims[i] for i in perm], [np.require(np.transpose(s, perm), requirements="C").copy() for s in x.slices])
