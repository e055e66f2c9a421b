"""TEST INFRASTRUCTURE.  Processor mesh, computation layout and per-processor slices.

Section 2 / Section 4: a mesh is an n-dimensional array of processors with named dimensions.
Section 4: a computation layout is a partial map tensor-dimension name -> mesh-dimension name.
Section 5: a tensor's layout is the restriction of that map to the tensor's dimensions and must be
injective (two dimensions of one tensor may not map to one mesh dimension); along every mapped
dimension a processor keeps the stripe selected by its coordinate on the mesh dimension; the
dimension size must be divisible by the mesh-dimension size; a tensor with an empty layout is fully
replicated.

Readings where the paper is silent: the stripe is a contiguous block (the slice shapes b/n x d_io
etc. of Section 8 fit this), and processor p has mesh coordinates obtained by row-major unranking
with the LAST mesh dimension varying fastest.
"""
from __future__ import annotations

import numpy as np

from .named import (DuplicateDim, IllegalLayout, NotDivisible, OracleError, UnknownDim, check_dims)


class Mesh:
    def __init__(self, dims):
        self.dims = check_dims(dims)
        self.names = tuple(n for n, _ in self.dims)
        self.shape = tuple(s for _, s in self.dims)
        self.P = int(np.prod(self.shape, dtype=np.int64)) if self.shape else 1

    def coords(self, p):
        """Mesh coordinates of processor p: p = sum_j c_j * prod_{j' > j} m_{j'}."""
        if not 0 <= p < self.P:
            raise OracleError(f"processor {p} outside mesh of {self.P}")
        c = []
        for m in reversed(self.shape):
            c.append(p % m)
            p //= m
        return tuple(reversed(c))

    def rank(self, coords):
        p = 0
        for c, m in zip(coords, self.shape):
            p = p * m + c
        return p

    def group(self, p, over):
        """Processors that agree with p on every mesh dimension NOT in ``over`` (a set of mesh-dim
        indices), in ascending processor order.  This is the group of a partitioned Allreduce."""
        cp = self.coords(p)
        out = []
        for q in range(self.P):
            cq = self.coords(q)
            if all(cq[j] == cp[j] for j in range(len(self.shape)) if j not in over):
                out.append(q)
        return out


class Layout:
    """A computation layout on a mesh: rules ((tensor_dim_name, mesh_dim_name), ...)."""

    def __init__(self, mesh, rules):
        self.mesh = mesh
        self.rules = {}
        for t, m in rules:
            if m not in mesh.names:
                raise UnknownDim(f"layout names mesh dimension {m!r}; mesh has {mesh.names}")
            if t in self.rules:
                raise OracleError(f"tensor dimension {t!r} is mapped twice (a layout is a map)")
            self.rules[t] = mesh.names.index(m)

    def mesh_dim_of(self, tdim_name):
        """Index of the mesh dimension a tensor dimension is split over, or None."""
        return self.rules.get(tdim_name)

    def tensor_layout(self, dims):
        """Restriction of the layout to ``dims``: {position in dims: mesh-dim index}.  Raises when
        it is not injective or a size is not divisible."""
        dims = check_dims(dims)
        used = {}
        out = {}
        for i, (n, s) in enumerate(dims):
            j = self.rules.get(n)
            if j is None:
                continue
            if j in used:
                raise IllegalLayout(
                    f"dimensions {used[j]!r} and {n!r} of one tensor are both split over mesh dimension "
                    f"{self.mesh.names[j]!r}")
            used[j] = n
            if s % self.mesh.shape[j] != 0:
                raise NotDivisible(f"dimension {n!r} of size {s} over mesh dimension of size {self.mesh.shape[j]}")
            out[i] = j
        return out

    def check_iteration_space(self, dim_lists):
        """Reading for an operation with several operands: the layout restricted to the union of all
        its dimensions must be injective as well, otherwise each processor would only see matching
        ("diagonal") blocks of two different split dimensions."""
        from .named import union_dims
        self.tensor_layout(union_dims(dim_lists))

    def slice_box(self, dims, p):
        """(offsets, sizes) of processor p's slice of a tensor with ``dims``."""
        tl = self.tensor_layout(dims)
        c = self.mesh.coords(p)
        offs, sizes = [], []
        for i, (_, s) in enumerate(dims):
            if i in tl:
                m = self.mesh.shape[tl[i]]
                t = s // m
                offs.append(c[tl[i]] * t)
                sizes.append(t)
            else:
                offs.append(0)
                sizes.append(s)
        return offs, sizes

    def slice_dims(self, dims, p=0):
        _, sizes = self.slice_box(dims, p)
        return tuple((n, t) for (n, _), t in zip(dims, sizes))

    def slice_of(self, dims, a, p):
        offs, sizes = self.slice_box(dims, p)
        idx = tuple(slice(o, o + t) for o, t in zip(offs, sizes))
        return np.require(a[idx], requirements="C").copy()

    def global_flat_indices(self, dims, p):
        """Flat row-major global index of every element of p's slice, in the slice's own row-major
        order: local l -> sum_i (o_i + l_i) * prod_{i' > i} s_{i'}."""
        offs, sizes = self.slice_box(dims, p)
        full = [s for _, s in dims]
        strides = [1] * len(full)
        for i in range(len(full) - 2, -1, -1):
            strides[i] = strides[i + 1] * full[i + 1]
        out = np.zeros(sizes, dtype=np.int64) if sizes else np.zeros((), dtype=np.int64)
        for i, (o, t) in enumerate(zip(offs, sizes)):
            shape = [1] * len(sizes)
            shape[i] = t
            out = out + ((o + np.arange(t, dtype=np.int64)) * strides[i]).reshape(shape)
        return out.reshape(-1)

    def split_mesh_dims(self, dims):
        """Mesh-dimension indices over which a tensor with ``dims`` is split."""
        return sorted(self.tensor_layout(dims).values())
