"""Pins of the oracle parts that go beyond the einsum and the blocks: the general rename of
Section 6.1 (Allgather / slice / Alltoall), the vocab-split embedding, logits and cross-entropy, the
parameter update of Algorithm 1 line 3, and the layout search over Table 1's cost counts."""
import itertools

import numpy as np
import pytest

import seeded_inputs as si
from oracle import NT, DenseOps, Layout, LoweredOps, Mesh, chooser, cost, update, vocab
from oracle.named import OracleError

dense = DenseOps()


def all_layouts(mesh_dims, names):
    return list(chooser.enumerate_layouts(mesh_dims, names))


# ---- Section 6.1: rename with a change of layout -----------------------------------------------------------

@pytest.mark.parametrize("mesh_dims", [[("a", 2)], [("a", 2), ("b", 3)], [("a", 2), ("b", 2), ("c", 2)]])
def test_reshape_every_layout_gives_the_dense_tensor_and_the_named_pattern(mesh_dims):
    # x[p, q, r] is reshaped to [p2, z, r]: two names change at once, so a mesh dimension can move from
    # one tensor dimension to another (the Alltoall case)
    dims = [("p", 12), ("q", 6), ("r", 12)]
    out_names = ["p2", "z", "r"]
    x = NT(dims, si.small_integers(5, "x", [12, 6, 12]))
    seen = set()
    checked = 0
    for rules in all_layouts(mesh_dims, ["p", "q", "r", "p2", "z"]):
        lay = Layout(Mesh(mesh_dims), rules)
        try:
            lay.tensor_layout(dims)
            lay.tensor_layout([("p2", 12), ("z", 6), ("r", 12)])
        except OracleError:
            continue
        ops = LoweredOps(lay)
        out = ops.reshape(ops.lower(x), out_names)
        got = ops.to_global(out)                       # also asserts that replicas are bitwise equal
        assert got.names == tuple(out_names) and np.array_equal(got.a, x.a)
        # per mesh dimension the pattern follows from which tensor POSITION is split before / after
        r = dict(rules)
        want = []
        for j, (m, _) in enumerate(mesh_dims):
            b_pos = next((i for i, (n, _) in enumerate(dims) if r.get(n) == m), None)
            a_pos = next((i for i, n in enumerate(out_names) if r.get(n) == m), None)
            if b_pos == a_pos:
                continue
            want.append((j, "allgather" if a_pos is None else "slice" if b_pos is None else "alltoall"))
        assert sorted((j, pat) for j, pat, _ in ops.reshape_log) == sorted(want), (rules, ops.reshape_log)
        seen |= {pat for _, pat in want}
        checked += 1
    assert checked >= 8 and seen == {"allgather", "slice", "alltoall"}


def test_reshape_communication_counts():
    # x[p=8, q=4] with q -> mesh dim of size 4, renamed to z (not split): Allgather, every processor
    # receives the other three stripes = 3 * 8 elements; the reverse is a local slice
    mesh = [("a", 4)]
    x = NT([("p", 8), ("q", 4)], si.small_integers(6, "x", [8, 4]))
    ops = LoweredOps(Layout(Mesh(mesh), [("q", "a")]))
    ops.rename(ops.lower(x), "q", "z")
    assert ops.reshape_log == [(0, "allgather", 24)]
    ops = LoweredOps(Layout(Mesh(mesh), [("z", "a")]))
    ops.rename(ops.lower(x), "q", "z")
    assert ops.reshape_log == [(0, "slice", 0)]
    # [p, q] with p -> a becomes [p2, z] with z -> a (the switch between a batch split and a model split
    # that Section 6.1 mentions): Alltoall, every processor keeps 1/4 of its 2 x 4 stripe and receives
    # 3/4 of a stripe's worth of elements
    ops = LoweredOps(Layout(Mesh(mesh), [("p", "a"), ("z", "a")]))
    out = ops.reshape(ops.lower(x), ["p2", "z"])
    assert ops.reshape_log == [(0, "alltoall", 6)]
    assert [s.shape for s in out.slices] == [(8, 1)] * 4
    assert np.array_equal(ops.to_global(out).a, x.a)
    assert np.array_equal(dense.reshape(x, ["p2", "z"]).a, x.a)


def test_transpose_is_local():
    x = NT([("b", 4), ("l", 6), ("h", 2), ("k", 3)], si.small_integers(7, "x", [4, 6, 2, 3]))
    lay = Layout(Mesh([("a", 2), ("c", 2)]), [("b", "a"), ("h", "c")])
    ops = LoweredOps(lay)
    out = ops.to_global(ops.transpose(ops.lower(x), ["b", "h", "l", "k"]))
    assert np.array_equal(out.a, np.transpose(x.a, (0, 2, 1, 3)))
    assert np.array_equal(dense.transpose(x, ["k", "b", "l", "h"]).a, np.transpose(x.a, (3, 0, 1, 2)))


# ---- vocab: embedding, logits, cross-entropy -----------------------------------------------------------------

def vocab_case(seed, B=2, L=3, D=4, V=6):
    tok = [("batch", B), ("length", L)]
    rng = np.random.RandomState(seed)
    ids, tgt = rng.randint(0, V, size=(B, L)), rng.randint(0, V, size=(B, L))
    E = NT([("vocab", V), ("d_model", D)], si.normal(seed, "E", [V, D], "f32").f64)
    wout = NT([("d_model", D), ("vocab", V)], si.normal(seed, "wo", [D, V], "f32", D ** -0.5).f64)
    dloss = NT(tok, np.full((B, L), 1.0 / (B * L)))
    return tok, ids, tgt, E, wout, dloss


def test_loss_is_minus_log_softmax_of_the_target_and_embedding_is_a_row_lookup():
    tok, ids, tgt, E, wout, _ = vocab_case(1)
    x = vocab.embedding_forward(dense, vocab.one_hot(ids, tok, E.dims[0]), E)
    assert np.array_equal(x.a, E.a[ids])
    f = vocab.xent_forward(dense, x, wout, vocab.one_hot(tgt, tok, E.dims[0]))
    lg = x.a @ wout.a
    p = np.exp(lg) / np.exp(lg).sum(-1, keepdims=True)
    want = -np.log(np.take_along_axis(p, tgt[..., None], -1))[..., 0]
    assert np.allclose(f["loss"].a, want, rtol=1e-12, atol=1e-12)
    # shifting a row of logits by a constant changes neither the loss nor the gradient (max subtraction)
    big = NT(x.dims, x.a * 50.0)
    assert np.isfinite(vocab.xent_forward(dense, big, wout, vocab.one_hot(tgt, tok, E.dims[0]))["loss"].a).all()


def test_cross_entropy_gradients_by_finite_differences():
    tok, ids, tgt, E, wout, dloss = vocab_case(2)
    oh_i, oh_t = vocab.one_hot(ids, tok, E.dims[0]), vocab.one_hot(tgt, tok, E.dims[0])

    def total(Ea, Wa):
        x = vocab.embedding_forward(dense, oh_i, NT(E.dims, Ea))
        return float((vocab.xent_forward(dense, x, NT(wout.dims, Wa), oh_t)["loss"].a * dloss.a).sum())

    x = vocab.embedding_forward(dense, oh_i, E)
    f = vocab.xent_forward(dense, x, wout, oh_t)
    g = vocab.xent_backward(dense, x, wout, f["logits"], f["lse"], oh_t, dloss)
    dE = vocab.embedding_backward(dense, oh_i, g["dh"], E.names)
    assert np.allclose(g["dlogits"].a.sum(-1), 0.0, atol=1e-15)          # softmax minus one-hot sums to zero
    eps = 1e-6
    for name, base, grad in (("E", E.a, dE.a), ("wout", wout.a, g["dwout"].a)):
        num = np.zeros_like(base)
        for idx in itertools.product(*[range(s) for s in base.shape]):
            hi, lo = base.copy(), base.copy()
            hi[idx] += eps
            lo[idx] -= eps
            num[idx] = ((total(hi, wout.a) if name == "E" else total(E.a, hi)) - (total(lo, wout.a) if name == "E" else total(E.a, lo))) / (2 * eps)
        assert np.allclose(grad, num, rtol=1e-6, atol=1e-8), name


@pytest.mark.parametrize("mesh_dims", [[("all", 2)], [("rows", 2), ("cols", 3)]])
def test_vocab_split_lowering_equals_dense_for_every_layout(mesh_dims):
    tok, ids, tgt, E, wout, dloss = vocab_case(3, B=2, L=2, D=4, V=6)
    oh_i, oh_t = vocab.one_hot(ids, tok, E.dims[0]), vocab.one_hot(tgt, tok, E.dims[0])
    x = vocab.embedding_forward(dense, oh_i, E)
    f = vocab.xent_forward(dense, x, wout, oh_t)
    g = vocab.xent_backward(dense, x, wout, f["logits"], f["lse"], oh_t, dloss)
    dE = vocab.embedding_backward(dense, oh_i, g["dh"], E.names)
    n_vocab_split = 0
    for rules in all_layouts(mesh_dims, ["batch", "vocab", "d_model"]):
        lay = Layout(Mesh(mesh_dims), rules)
        try:
            for d in (oh_i.dims, E.dims, wout.dims, x.dims):
                lay.tensor_layout(d)
        except OracleError:
            continue
        ops = LoweredOps(lay)
        low = {k: ops.lower(t) for k, t in dict(oh_i=oh_i, oh_t=oh_t, E=E, wout=wout, dloss=dloss).items()}
        lx = vocab.embedding_forward(ops, low["oh_i"], low["E"])
        lf = vocab.xent_forward(ops, lx, low["wout"], low["oh_t"])
        lb = vocab.xent_backward(ops, lx, low["wout"], lf["logits"], lf["lse"], low["oh_t"], low["dloss"])
        lE = vocab.embedding_backward(ops, low["oh_i"], lb["dh"], E.names)
        for got, want in ((lx, x), (lf["loss"], f["loss"]), (lf["lse"], f["lse"]), (lb["dh"], g["dh"]), (lb["dwout"], g["dwout"]), (lE, dE)):
            assert np.allclose(ops.to_global(got).a, want.a, rtol=1e-12, atol=1e-13), rules
        if dict(rules).get("vocab") is not None:
            n_vocab_split += 1
            j = lay.mesh_dim_of("vocab")
            tags = [(tag, over) for tag, over, _ in ops.allreduce_log if j in over]
            # the embedding lookup, the row maximum, the row sum of exponentials, the picked logit and dh all
            # reduce out `vocab`: each needs its Allreduce over the mesh dimension vocab is split over
            assert [t for t, _ in tags].count("reduce_max") == 1 and [t for t, _ in tags].count("reduce_sum") == 2
            assert [t for t, _ in tags].count("einsum") >= 2
    assert n_vocab_split >= 1


# ---- Algorithm 1 line 3 ------------------------------------------------------------------------------------------

def test_update_closed_forms():
    w0 = si.normal(4, "w", [5, 7], "f32").f64
    g = si.normal(4, "g", [5, 7], "f32").f64
    lr, mu, wd, n = 0.1, 0.9, 0.01, 6
    w, m = w0.copy(), None
    for _ in range(n):                                   # plain SGD: W_n = W_0 - n lr g
        w, m = update.sgd_update(w, g, None, lr)
    assert np.allclose(w, w0 - n * lr * g, rtol=1e-13) and m is None
    w, m = w0.copy(), np.zeros_like(w0)
    for _ in range(n):                                   # momentum with a constant gradient: m_k = g (1 - mu^k) / (1 - mu)
        w, m = update.sgd_update(w, g, m, lr, mu)
    assert np.allclose(m, g * (1 - mu ** n) / (1 - mu), rtol=1e-12)
    assert np.allclose(w, w0 - lr * g * sum((1 - mu ** k) / (1 - mu) for k in range(1, n + 1)), rtol=1e-12)
    w = w0.copy()
    for _ in range(n):                                   # weight decay alone: W_n = W_0 (1 - lr wd)^n
        w, _ = update.sgd_update(w, np.zeros_like(g), None, lr, 0.0, wd)
    assert np.allclose(w, w0 * (1 - lr * wd) ** n, rtol=1e-13)


def test_update_is_local_under_every_layout():
    dims = [("d_model", 4), ("d_ff", 6)]
    w, g, m = (NT(dims, si.small_integers(8, k, [4, 6])) for k in "wgm")
    want, want_m = update.sgd_update(w.a, g.a, m.a, 0.5, 0.25, 0.125)
    for rules in all_layouts([("a", 2), ("b", 3)], ["d_model", "d_ff"]):
        lay = Layout(Mesh([("a", 2), ("b", 3)]), rules)
        try:
            lay.tensor_layout(dims)
        except OracleError:
            continue
        ops = LoweredOps(lay)
        new, new_m = update.lowered_update(ops, ops.lower(w), ops.lower(g), ops.lower(m), 0.5, 0.25, 0.125)
        assert np.array_equal(ops.to_global(new).a, want) and np.array_equal(ops.to_global(new_m).a, want_m)   # (powers of two: exact)
        assert ops.allreduce_log == []


# ---- layout search over Table 1 ------------------------------------------------------------------------------------

def fc_einsums(b, d_io, d_h):
    x, w, v = [("batch", b), ("io", d_io)], [("io", d_io), ("hidden", d_h)], [("hidden", d_h), ("io", d_io)]
    h = [("batch", b), ("hidden", d_h)]
    return [([x, w], ["batch", "hidden"]), ([h, v], ["batch", "io"]),                      # forward
            ([x, v], ["batch", "hidden"]), ([h, x], ["hidden", "io"]), ([x, h], ["io", "hidden"]), ([h, w], ["batch", "io"])]   # backward


def test_search_agrees_with_table_1_on_one_mesh_dimension():
    # Table 1, n processors: data-parallel communicates ~ d_io d_h values, model-parallel ~ b d_io; both divide
    # the computation by n.  So with one mesh dimension the search must pick the batch split when b > d_h and
    # the hidden split when d_h > b (comm_weight > 0), and nothing is cheaper than either.
    n = 4
    for b, d_h, want in ((64, 16, "batch"), (16, 64, "hidden")):
        rules, c, _ = chooser.choose_layout([("all", n)], ["batch", "hidden", "io"], fc_einsums(b, 8, d_h), comm_weight=4.0)
        assert rules == [(want, "all")], (b, d_h, rules)
        # its cost is the table's: computation 6 b d_io d_h / n multiply-adds ...
        comp = 6 * b * 8 * d_h // n
        comm = c - comp
        # ... plus the Allreduced values: 2 d_io d_h (data-parallel: dw and dv) or 2 b d_io (model-parallel: y and dx)
        assert comm == 4.0 * (2 * 8 * d_h if want == "batch" else 2 * b * 8)


def test_search_finds_the_two_dimensional_layout_of_section_8_3():
    # r x c mesh: splitting batch over one mesh dimension and hidden over the other divides the computation
    # by r c; every one-dimensional choice leaves a factor on the table
    rules, _, _ = chooser.choose_layout([("rows", 2), ("cols", 4)], ["batch", "hidden", "io"], fc_einsums(32, 8, 32), comm_weight=1.0)
    assert sorted(rules) in ([("batch", "cols"), ("hidden", "rows")], [("batch", "rows"), ("hidden", "cols")])
    # zero communication weight and a tie in computation: the smaller footprint wins
    rules0, c0, _ = chooser.choose_layout([("rows", 2), ("cols", 4)], ["batch", "hidden", "io"], fc_einsums(32, 8, 32), comm_weight=0.0)
    assert c0 == 6 * 32 * 8 * 32 // 8
