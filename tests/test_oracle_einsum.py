"""Pins for the oracle's einsum loop nest and dense ops (CPU only).

The loop nest is tied to things other than itself:
  * a literal reading of the definition in Section 6 (broadcast every input to the union of all
    dimensions, multiply, sum out what is not in the output), done here with numpy broadcasting;
  * the matrix / batched-matrix special cases, which must equal numpy's matmul;
  * algebraic invariants (linearity, output-order transposition, trace and outer product).
"""
import itertools

import numpy as np
import pytest

from oracle import NT, DenseOps, DuplicateDim, SizeMismatch, UnknownDim, einsum_arrays
import seeded_inputs as si


def brute_force(in_dims, arrays, out_names):
    """Materialise the broadcast product over the union of dims, then reduce (numpy only)."""
    union = []
    for d in in_dims:
        for n, s in d:
            if n not in [u for u, _ in union]:
                union.append((n, s))
    names = [n for n, _ in union]
    prod = np.ones([s for _, s in union])
    for d, a in zip(in_dims, arrays):
        dn = [n for n, _ in d]
        perm = [dn.index(n) for n in names if n in dn]
        shape = [s if n in dn else 1 for n, s in union]
        prod = prod * np.transpose(a, perm).reshape(shape)
    axes = tuple(i for i, n in enumerate(names) if n not in out_names)
    r = prod.sum(axis=axes) if axes else prod
    rem = [n for n in names if n in out_names]
    return np.transpose(r, [rem.index(n) for n in out_names])


CASES = [
    ([[("i", 3), ("k", 4)], [("k", 4), ("j", 5)]], ["i", "j"]),
    ([[("i", 3), ("k", 4)], [("k", 4), ("j", 5)]], ["j", "i"]),
    ([[("i", 3), ("k", 4)], [("j", 5), ("k", 4)]], ["i", "j"]),
    ([[("b", 2), ("i", 3), ("k", 4)], [("b", 2), ("k", 4), ("j", 5)]], ["b", "i", "j"]),
    ([[("b", 2), ("l", 3), ("h", 2), ("k", 4)], [("b", 2), ("m", 5), ("h", 2), ("k", 4)]], ["b", "h", "l", "m"]),
    ([[("b", 2), ("l", 3), ("d", 4)], [("d", 4), ("h", 2), ("k", 3)]], ["b", "l", "h", "k"]),
    ([[("i", 3), ("k", 4)]], ["i"]),                       # one operand: a reduction
    ([[("i", 3), ("k", 4)]], ["k", "i"]),                  # one operand: a transpose
    ([[("i", 3), ("k", 4)]], []),                          # full reduction
    ([[("i", 3)], [("j", 4)]], ["i", "j"]),                # outer product (pure broadcast)
    ([[("i", 3), ("k", 4)], [("k", 4), ("j", 5)], [("j", 5), ("l", 2)]], ["i", "l"]),   # three operands
    ([[("i", 3), ("k", 4)], [("k", 4)], [("i", 3)]], ["i"]),
    ([[("i", 3), ("p", 2), ("k", 4)], [("k", 4), ("j", 5)]], ["i", "j"]),  # private reduced dim p
]


@pytest.mark.parametrize("in_dims,out_names", CASES)
def test_loop_nest_equals_literal_definition(in_dims, out_names):
    arrays = [si.normal_f64(7, f"e{q}", int(np.prod([s for _, s in d]))).reshape([s for _, s in d])
              for q, d in enumerate(in_dims)]
    got = einsum_arrays(in_dims, arrays, out_names)
    want = brute_force(in_dims, arrays, out_names)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-13)


def test_matrix_special_cases_equal_numpy_matmul():
    a = si.normal_f64(1, "a", 7 * 9).reshape(7, 9)
    b = si.normal_f64(1, "b", 9 * 5).reshape(9, 5)
    np.testing.assert_allclose(einsum_arrays([[("i", 7), ("k", 9)], [("k", 9), ("j", 5)]], [a, b], ["i", "j"]),
                               a @ b, rtol=1e-13, atol=1e-13)
    # transposed operand: A[i,k] . B[j,k] -> A @ B^T
    bt = np.ascontiguousarray(b.T)
    np.testing.assert_allclose(einsum_arrays([[("i", 7), ("k", 9)], [("j", 5), ("k", 9)]], [a, bt], ["i", "j"]),
                               a @ b, rtol=1e-13, atol=1e-13)
    # reduce over the slow dim of both operands: A[k,i] . B[k,j] -> A^T @ B
    at = np.ascontiguousarray(a.T)
    np.testing.assert_allclose(einsum_arrays([[("k", 9), ("i", 7)], [("k", 9), ("j", 5)]], [at, b], ["i", "j"]),
                               a @ b, rtol=1e-13, atol=1e-13)
    # batched
    A = si.normal_f64(2, "A", 3 * 4 * 6).reshape(3, 4, 6)
    B = si.normal_f64(2, "B", 3 * 6 * 2).reshape(3, 6, 2)
    np.testing.assert_allclose(
        einsum_arrays([[("b", 3), ("i", 4), ("k", 6)], [("b", 3), ("k", 6), ("j", 2)]], [A, B], ["b", "i", "j"]),
        np.matmul(A, B), rtol=1e-13, atol=1e-13)


def test_exact_on_small_integers_and_identity():
    a = si.small_integers(3, "ia", (6, 8))
    eye = np.eye(8)
    got = einsum_arrays([[("i", 6), ("k", 8)], [("k", 8), ("j", 8)]], [a, eye], ["i", "j"])
    assert np.array_equal(got, a)
    # trace-like full contraction equals the Frobenius inner product
    b = si.small_integers(3, "ib", (6, 8))
    got = einsum_arrays([[("i", 6), ("k", 8)], [("i", 6), ("k", 8)]], [a, b], [])
    assert got.shape == () and float(got) == float((a * b).sum())


def test_linearity_in_each_operand():
    d = [[("i", 4), ("k", 5)], [("k", 5), ("j", 3)]]
    a1, a2 = si.small_integers(4, "a1", (4, 5)), si.small_integers(4, "a2", (4, 5))
    b = si.small_integers(4, "b", (5, 3))
    lhs = einsum_arrays(d, [2 * a1 - 3 * a2, b], ["i", "j"])
    rhs = 2 * einsum_arrays(d, [a1, b], ["i", "j"]) - 3 * einsum_arrays(d, [a2, b], ["i", "j"])
    assert np.array_equal(lhs, rhs)


def test_errors():
    ops = DenseOps()
    with pytest.raises(DuplicateDim):
        NT([("i", 2), ("i", 2)], np.zeros((2, 2)))
    a = NT([("i", 2), ("k", 3)], np.zeros((2, 3)))
    b = NT([("k", 4), ("j", 2)], np.zeros((4, 2)))
    with pytest.raises(SizeMismatch):
        ops.einsum([a, b], ["i", "j"])
    c = NT([("k", 3), ("j", 2)], np.zeros((3, 2)))
    with pytest.raises(UnknownDim):
        ops.einsum([a, c], ["i", "z"])


def test_broadcast_binary_and_reductions_match_numpy():
    ops = DenseOps()
    x = NT([("b", 3), ("h", 4)], si.normal_f64(5, "x", 12).reshape(3, 4))
    bias = NT([("h", 4)], si.normal_f64(5, "bias", 4))
    np.testing.assert_array_equal(ops.add(x, bias).a, x.a + bias.a[None, :])
    np.testing.assert_array_equal(ops.add(bias, x).a, x.a + bias.a[None, :])
    col = NT([("b", 3)], si.normal_f64(5, "col", 3))
    np.testing.assert_array_equal(ops.sub(x, col).a, x.a - col.a[:, None])
    np.testing.assert_array_equal(ops.reduce_sum(x, ["h"]).a, x.a.sum(0))
    np.testing.assert_array_equal(ops.reduce_max(x, ["b"]).a, x.a.max(1))
    np.testing.assert_array_equal(ops.relu(x).a, np.where(x.a > 0, x.a, 0.0))
    # a reduction is the one-operand einsum
    np.testing.assert_allclose(ops.reduce_sum(x, ["b"]).a, ops.einsum([x], ["b"]).a, rtol=1e-14)
