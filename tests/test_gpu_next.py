"""GPU parity of the rows beyond the blocks, through the C ABI against the oracle: the parameter
update of Algorithm 1 line 3, the storage-order and slice copies of Section 6.1 (bit-exact), and the
vocab dimension of the Section 9 layout - embedding lookup (bit-exact), its gradient, and the logits
einsum with softmax cross-entropy, forward and backward, checked launch by launch."""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import TOL, Guarded, from_torch, parity_error, to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mtf():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1811_02084_b200 as m
    return m


def layout(mtf, mesh_dims, rules):
    return mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules)


# ---- Algorithm 1 line 3 ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("shape", [(256, 512), (37, 41), (3,), (1024, 1030)], ids=str)       # whole vectors, ragged tails, tiny
@pytest.mark.parametrize("grad_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("with_momentum", [False, True])
def test_update_matches_oracle(mtf, shape, grad_dtype, with_momentum):
    import torch
    from oracle import update
    dims = list(zip(["d_model", "d_ff"], shape))
    names = [n for n, _ in dims]
    w0, g, m0 = si.normal(30, "w", shape, "f32"), si.normal(30, "g", shape, grad_dtype), si.normal(30, "m", shape, "f32", 0.5)
    lr, mu, wd = 0.05, 0.9 if with_momentum else 0.0, 0.01
    guard = Guarded()
    w, mom, wb = guard.empty(shape, "f32"), guard.empty(shape, "f32"), guard.empty(shape, "bf16")
    w.copy_(to_torch(w0)); mom.copy_(to_torch(m0))
    gt = to_torch(g)
    lay = layout(mtf, [("all", 1)], []) if len(shape) == 1 or shape[1] % 2 else layout(mtf, [("all", 2)], [("d_ff", "all")])
    ref_w, ref_m = w0.f64, m0.f64 if with_momentum else None
    for _ in range(3):
        mtf.mtf_update(lay, mtf.named(gt, names), mtf.named(w, names), mtf.named(mom, names) if with_momentum else None, mtf.named(wb, names), lr, mu, wd)
        ref_w, ref_m = update.sgd_update(ref_w, g.f64, ref_m, lr, mu, wd)
    mtf.mtf_device_status()
    guard.check()
    assert parity_error(from_torch(w), ref_w) <= TOL["f32"]
    if with_momentum:
        assert parity_error(from_torch(mom), ref_m) <= TOL["f32"]
    else:
        assert np.array_equal(from_torch(mom), m0.f64)            # untouched
    # the working copy is the round-to-nearest-even bf16 of the GPU's own master values: bit-exact
    assert torch.equal(wb, w.to(torch.bfloat16))


# ---- Section 6.1: storage order and slices --------------------------------------------------------------------------

PERMS = [
    ([("batch", 3), ("length", 40), ("heads", 4), ("d_k", 64)], ["batch", "heads", "length", "d_k"], "bf16"),     # rows of 128 bytes move whole
    ([("batch", 3), ("heads", 4), ("length", 40), ("d_k", 64)], ["batch", "length", "heads", "d_k"], "bf16"),
    ([("batch", 2), ("length", 70), ("d_model", 136)], ["batch", "d_model", "length"], "bf16"),                      # the innermost dimension changes: tiles
    ([("a", 5), ("b", 33), ("c", 7), ("d", 66)], ["d", "b", "a", "c"], "f32"),
    ([("a", 130), ("b", 67)], ["b", "a"], "f32"),
    ([("a", 6), ("b", 10), ("c", 12)], ["b", "a", "c"], "f32"),                                                        # rows of 48 bytes
    ([("a", 6), ("b", 10), ("c", 5)], ["b", "a", "c"], "bf16"),                                                        # rows that are no multiple of 16 bytes
]


@pytest.mark.parametrize("dims,out_names,dtype", PERMS, ids=lambda p: str(p) if isinstance(p, str) else None)
def test_transpose_is_bit_exact(mtf, dims, out_names, dtype):
    import torch
    x = si.normal(31, "x", [s for _, s in dims], dtype)
    xt = to_torch(x)
    perm = [[n for n, _ in dims].index(n) for n in out_names]
    guard = Guarded()
    out = guard.empty([dims[i][1] for i in perm], dtype)
    lay = layout(mtf, [("all", 1)], [])
    mtf.mtf_transpose(lay, mtf.named(xt, [n for n, _ in dims]), mtf.named(out, out_names))
    mtf.mtf_device_status()
    guard.check()
    assert torch.equal(out, xt.permute(perm).contiguous())


def test_slice_gather_then_scatter_rebuilds_the_tensor(mtf):
    import torch
    from oracle import Layout, Mesh
    dims = [("batch", 4), ("length", 6), ("d_ff", 48)]
    mesh_dims, rules = [("rows", 2), ("cols", 3)], [("batch", "rows"), ("d_ff", "cols")]
    lay, olay = layout(mtf, mesh_dims, rules), Layout(Mesh(mesh_dims), rules)
    x = si.normal(32, "x", [4, 6, 48], "bf16")
    xt = to_torch(x)
    names = [n for n, _ in dims]
    guard = Guarded()
    rebuilt = guard.empty([4, 6, 48], "bf16")
    for p in range(6):
        _, sizes = olay.slice_box(dims, p)
        sl = guard.empty(sizes, "bf16")
        mtf.mtf_slice_gather(lay, mtf.named(xt, names), p, sl)
        assert np.array_equal(from_torch(sl), olay.slice_of(dims, x.f64, p))             # the Allgather's input: each processor's stripe
        mtf.mtf_slice_scatter(lay, sl, p, mtf.named(rebuilt, names))
    mtf.mtf_device_status()
    guard.check()
    assert torch.equal(rebuilt, xt)


# ---- vocab: embedding, logits, cross-entropy -----------------------------------------------------------------------

VOCAB_LAYOUTS = [([("all", 1)], []), ([("all", 4)], [("vocab", "all")]), ([("rows", 2), ("cols", 2)], [("batch", "rows"), ("vocab", "cols")])]


def vocab_case(seed, B, L, D, V):
    rng = np.random.RandomState(seed)
    ids, tgt = rng.randint(0, V, size=(B, L)).astype(np.int32), rng.randint(0, V, size=(B, L)).astype(np.int32)
    ids[0, 0], ids[-1, -1], tgt[0, 0], tgt[-1, -1] = 0, V - 1, V - 1, 0           # first and last rows / columns of every slice take part
    E = si.normal(seed, "E", [V, D], "bf16")
    wout = si.normal(seed, "wout", [D, V], "bf16", D ** -0.5)
    return ids, tgt, E, wout


def run_vocab_stagewise(mtf, lay, B, L, D, V, seed, tok=None, cols=None):
    """Embedding + logits + cross-entropy forward and backward, every launch against the exact oracle of that
    launch on the inputs the launch read.  tok / cols: sampled tokens / vocab columns (None = all)."""
    import torch
    from oracle import stages, vocab as ov
    from stagewise import StageReport, Tap, _idx, _nt
    ids, tgt, E, wout = vocab_case(seed, B, L, D, V)
    T = B * L
    tok = np.arange(T) if tok is None else np.asarray(tok)
    cols = np.arange(V) if cols is None else np.asarray(cols)
    guard = Guarded()
    ids_t, tgt_t = torch.from_numpy(ids).cuda(), torch.from_numpy(tgt).cuda()
    Et, Wt = to_torch(E), to_torch(wout)
    x, logits = guard.empty([B, L, D], "bf16"), guard.empty([B, L, V], "bf16")
    lse, loss, dloss = guard.empty([B, L], "f32"), guard.empty([B, L], "f32"), guard.empty([B, L], "f32")
    dh, dwout, dE = guard.empty([B, L, D], "bf16"), guard.empty([D, V], "f32"), guard.empty([V, D], "f32")
    dl = si.normal(seed, "dloss", [B, L], "f32", 1.0 / T, 1.0 / T)
    dloss.copy_(to_torch(dl))
    N = mtf.named
    act, lgn = ["batch", "length", "d_model"], ["batch", "length", "vocab"]
    ws = guard.empty([64 << 20], "u8")
    tap = Tap(mtf, T * V * 2 + 4096, guard)
    mtf.mtf_embedding_forward(lay, ids_t, N(Et, ["vocab", "d_model"]), N(x, act))
    mtf.mtf_xent_forward(lay, N(x, act), N(Wt, ["d_model", "vocab"]), tgt_t, N(logits, lgn), N(lse, ["batch", "length"]), N(loss, ["batch", "length"]), ws)
    lg_gpu = logits.clone()
    mtf.mtf_xent_backward(lay, N(x, act), N(Wt, ["d_model", "vocab"]), tgt_t, N(logits, lgn), N(lse, ["batch", "length"]), N(dloss, ["batch", "length"]),
                          N(dh, act), N(dwout, ["d_model", "vocab"]), ws)
    mtf.mtf_embedding_backward(lay, ids_t, N(dh, act), N(dE, ["vocab", "d_model"]))
    tap.close()
    mtf.mtf_device_status()
    guard.check()
    G = from_torch
    rep = StageReport(TOL["bf16"], "vocab")
    ti, ci = _idx(tok), _idx(cols)
    # the lookup is a copy: bit-exact, every row
    assert torch.equal(x.view(T, D), Et[torch.from_numpy(ids.reshape(-1).astype(np.int64)).cuda()])
    x_t = _nt(["t", "d"], G(x.view(T, D)[ti]))
    ref, _ = stages.contraction(x_t, _nt(["d", "v"], wout.f64), ["t", "v"])
    rep.add("logits", G(lg_gpu.view(T, V)[ti]), ref.a)
    # row statistics and loss from the logits the GPU stored (fp32 arithmetic: the fp32 tolerance)
    lg_rows = G(lg_gpu.view(T, V)[ti])
    mx = lg_rows.max(-1)
    lse_ref = mx + np.log(np.exp(lg_rows - mx[:, None]).sum(-1))
    tg = tgt.reshape(-1)[tok]
    rep.add("lse", G(lse.view(T)[ti]), lse_ref, tol=TOL["f32"])
    rep.add("loss", G(loss.view(T)[ti]), lse_ref - lg_rows[np.arange(len(tok)), tg], tol=TOL["f32"])
    # dlogits from the GPU's logits and the GPU's lse
    dlg_gpu = tap.get("dlogits", [T, V], "bf16")
    oh = (tg[:, None] == np.arange(V)).astype(np.float64)
    rep.add("dlogits", G(dlg_gpu[ti]), (np.exp(lg_rows - G(lse.view(T)[ti])[:, None]) - oh) * dl.f64.reshape(-1)[tok][:, None])
    # dh = dlogits . wout^T (reduces vocab) on sampled tokens; dwout = h^T . dlogits on sampled vocab columns, all tokens
    ref, _ = stages.contraction(_nt(["t", "v"], G(dlg_gpu[ti])), _nt(["d", "v"], wout.f64), ["t", "d"])
    rep.add("dh", G(dh.view(T, D)[ti]), ref.a)
    ref, _ = stages.contraction(_nt(["t", "d"], G(x.view(T, D))), _nt(["t", "v"], G(dlg_gpu[:, ci])), ["d", "v"])
    rep.add("dwout", G(dwout[:, ci]), ref.a)
    # dE[v, :] = sum of dh rows whose id is v (f32 atomics): against the oracle's one-hot einsum on the GPU's dh, sampled rows of the table
    vrows = np.unique(np.concatenate([ids.reshape(-1)[tok], [0, V - 1]]))
    oh_i = (ids.reshape(-1)[:, None] == vrows[None, :]).astype(np.float64)
    ref, _ = stages.contraction(_nt(["t", "v"], oh_i), _nt(["t", "d"], G(dh.view(T, D))), ["v", "d"])
    rep.add("dE", G(dE[_idx(vrows)]), ref.a, tol=TOL["f32"])
    return rep.finish()


@pytest.mark.parametrize("mesh_dims,rules", VOCAB_LAYOUTS)
def test_vocab_block_stagewise(mtf, mesh_dims, rules):
    errs = run_vocab_stagewise(mtf, layout(mtf, mesh_dims, rules), 4, 36, 128, 1000, 33)     # vocab 1000: slices of 250 columns, ragged tiles
    print(errs)


def test_vocab_full_size_stagewise(mtf):
    # vocab 32768, d_model 1024, tokens 8192 (batch 32 x length 256): sampled tokens and vocab columns
    B, L, D, V = 32, 256, 1024, 32768
    tok = si.sample_indices(0, "vtok", B * L, 6, must_include=[0, B * L - 1, L - 1, L, 16 * L - 1, 16 * L])
    cols = si.sample_indices(0, "vcol", V, 6, must_include=[0, V - 1, V // 4 - 1, V // 4, V // 2, 3 * V // 4 - 1])
    for mesh_dims, rules in (([("all", 8)], [("vocab", "all")]), ([("rows", 4), ("cols", 8)], [("batch", "rows"), ("vocab", "cols")])):
        errs = run_vocab_stagewise(mtf, layout(mtf, mesh_dims, rules), B, L, D, V, 34, tok, cols)
        print(rules, {k: f"{e:.2e}" for k, e in errs.items()})


def test_out_of_range_ids_are_reported(mtf):
    import torch
    lay = layout(mtf, [("all", 1)], [])
    E = to_torch(si.normal(35, "E", [16, 8], "bf16"))
    ids = torch.tensor([[0, 15, 16, -1]], dtype=torch.int32, device="cuda")
    x = torch.full((1, 4, 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    mtf.mtf_embedding_forward(lay, ids, mtf.named(E, ["vocab", "d_model"]), mtf.named(x, ["batch", "length", "d_model"]))
    with pytest.raises(mtf.MtfError) as e:
        mtf.mtf_device_status()
    assert e.value.code == "MTF_ERR_INVALID_ARG"
    assert torch.equal(x[0, :2], E[[0, 15]]) and bool((x[0, 2:] == 0).all())
    mtf.mtf_device_status()                                   # the flag was reset
