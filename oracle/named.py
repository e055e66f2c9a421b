"""TEST INFRASTRUCTURE.  Named-dimension tensors and the un-split ("dense") operations on them.

Follows Section 4 (tensors have named dimensions, no duplicate names in one tensor), Section 6
(component-wise operations, reductions, einsum by its plain definition) and Section 7 (a binary
component-wise operation broadcasts an operand whose shape is a subset of the other's).
Everything is fp64.
"""
from __future__ import annotations

import numpy as np

from . import _core


class OracleError(Exception):
    """Base class; ``code`` matches the name of the library's status code for the same mistake."""
    code = "MTF_ERR_INVALID_ARG"


class DuplicateDim(OracleError):
    code = "MTF_ERR_DUPLICATE_DIM"


class UnknownDim(OracleError):
    code = "MTF_ERR_UNKNOWN_DIM"


class SizeMismatch(OracleError):
    code = "MTF_ERR_SIZE_MISMATCH"


class IllegalLayout(OracleError):
    code = "MTF_ERR_ILLEGAL_LAYOUT"


class NotDivisible(OracleError):
    code = "MTF_ERR_NOT_DIVISIBLE"


def check_dims(dims):
    """Section 4: a tensor may not carry two identically named dimensions; sizes are static and positive."""
    names = [n for n, _ in dims]
    if len(set(names)) != len(names):
        raise DuplicateDim(f"duplicate dimension name in {names}")
    for n, s in dims:
        if int(s) <= 0:
            raise OracleError(f"dimension {n!r} has non-positive size {s}")
    return tuple((str(n), int(s)) for n, s in dims)


class NT:
    """A named tensor: ``dims`` = ((name, size), ...) in storage order, ``a`` = fp64 array of that shape."""

    __slots__ = ("dims", "a")

    def __init__(self, dims, a):
        self.dims = check_dims(dims)
        a = np.asarray(a, dtype=np.float64)
        if tuple(a.shape) != tuple(s for _, s in self.dims):
            raise SizeMismatch(f"array shape {a.shape} does not match dims {self.dims}")
        self.a = np.require(a, dtype=np.float64, requirements="C")

    @property
    def names(self):
        return tuple(n for n, _ in self.dims)

    def size_of(self, name):
        for n, s in self.dims:
            if n == name:
                return s
        raise UnknownDim(name)

    def __repr__(self):
        return f"NT({self.dims})"


def union_dims(dim_lists):
    """Union of named dims in first-seen order; the same name must have the same size everywhere."""
    seen = {}
    order = []
    for dims in dim_lists:
        for n, s in dims:
            if n in seen:
                if seen[n] != s:
                    raise SizeMismatch(f"dimension {n!r} has sizes {seen[n]} and {s}")
            else:
                seen[n] = s
                order.append((n, s))
    return order


def resolve_out_dims(in_dim_lists, out_names):
    """Output dims must be a subset of the union of the input dims (sizes taken from the inputs)."""
    u = dict(union_dims(in_dim_lists))
    out = []
    for item in out_names:
        n, s = (item, None) if isinstance(item, str) else item
        if n not in u:
            raise UnknownDim(f"output dimension {n!r} is in no input")
        if s is not None and int(s) != u[n]:
            raise SizeMismatch(f"output dimension {n!r} has size {s}, inputs have {u[n]}")
        out.append((n, u[n]))
    return check_dims(out)


def einsum_arrays(in_dims, in_arrays, out_dims):
    """Plain-definition einsum on raw fp64 arrays (Section 6).  Returns the output array."""
    in_dims = [check_dims(d) for d in in_dims]
    out_dims = resolve_out_dims(in_dims, out_dims)
    u = union_dims(in_dims)
    out_names = [n for n, _ in out_dims]
    red = [(n, s) for n, s in u if n not in out_names]
    space = list(out_dims) + red                      # iteration space: output dims, then reduced dims
    sizes = [s for _, s in space]
    in_strides = []
    arrays = []
    for dims, a in zip(in_dims, in_arrays):
        a = np.require(a, dtype=np.float64, requirements="C")
        elem_strides = {n: st // 8 for (n, _), st in zip(dims, a.strides)} if a.ndim else {}
        in_strides.append([elem_strides.get(n, 0) for n, _ in space])
        arrays.append(a)
    out = np.zeros([s for _, s in out_dims], dtype=np.float64)
    out_strides = [st // 8 for st in out.strides]
    _core.einsum_loops(sizes, in_strides, out_strides, len(out_dims), arrays, out)
    return out


class DenseOps:
    """The un-split computation: every operation acts on whole tensors."""

    def einsum(self, inputs, out_names):
        out_dims = resolve_out_dims([t.dims for t in inputs], out_names)
        return NT(out_dims, einsum_arrays([t.dims for t in inputs], [t.a for t in inputs], out_dims))

    # -- component-wise (Section 6) and broadcasting binary ops (Section 7) -----------------------
    @staticmethod
    def _expand(small, big):
        """View of ``small`` broadcast against ``big``; small's dim names must be a subset of big's."""
        for n, s in small.dims:
            if n not in big.names:
                raise UnknownDim(f"cannot broadcast: {n!r} not in {big.names}")
            if big.size_of(n) != s:
                raise SizeMismatch(n)
        # order small's axes as they appear in big, then insert length-1 axes
        order = [small.names.index(n) for n in big.names if n in small.names]
        a = np.transpose(small.a, order) if order else small.a
        shape = [s if n in small.names else 1 for n, s in big.dims]
        return a.reshape(shape)

    def _binary(self, x, y, fn):
        if len(y.dims) > len(x.dims):
            return NT(y.dims, fn(self._expand(x, y), y.a))
        return NT(x.dims, fn(x.a, self._expand(y, x)))

    def add(self, x, y):
        return self._binary(x, y, np.add)

    def sub(self, x, y):
        return self._binary(x, y, np.subtract)

    def mul(self, x, y):
        return self._binary(x, y, np.multiply)

    def unary(self, x, fn):
        return NT(x.dims, fn(x.a))

    def relu(self, x):
        return self.unary(x, lambda a: np.maximum(a, 0.0))

    def positive(self, x):
        """Indicator [x > 0]; the derivative of relu with relu'(0) = 0."""
        return self.unary(x, lambda a: (a > 0.0).astype(np.float64))

    def exp(self, x):
        return self.unary(x, np.exp)

    def scale(self, x, c):
        return self.unary(x, lambda a: a * float(c))

    def rsqrt_plus(self, x, eps):
        return self.unary(x, lambda a: 1.0 / np.sqrt(a + eps))

    # -- reductions (Section 6) ---------------------------------------------------------------------
    def _reduce(self, x, out_names, fn):
        out_dims = resolve_out_dims([x.dims], out_names)
        keep = [n for n, _ in out_dims]
        axes = tuple(i for i, n in enumerate(x.names) if n not in keep)
        r = fn(x.a, axis=axes) if axes else x.a.copy()
        rem = [n for n in x.names if n in keep]
        r = np.transpose(r, [rem.index(n) for n in keep]) if keep else r
        return NT(out_dims, r)

    def reduce_sum(self, x, out_names):
        return self._reduce(x, out_names, np.sum)

    def reduce_max(self, x, out_names):
        return self._reduce(x, out_names, np.max)

    def rename(self, x, old, new):
        """Same data, one dimension renamed (a reshape that changes only a name)."""
        return NT([(new if n == old else n, s) for n, s in x.dims], x.a)

    def reshape(self, x, out_names):
        """Same data, dimensions renamed position by position (sizes kept)."""
        return NT([(n, s) for n, (_, s) in zip(out_names, x.dims)], x.a)

    def transpose(self, x, out_names):
        """Same dimensions in another storage order."""
        perm = [x.names.index(n) for n in out_names]
        return NT([x.dims[i] for i in perm], np.transpose(x.a, perm))

    def to_global(self, x):
        return x

    def lower(self, x):
        return x
