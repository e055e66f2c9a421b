"""Stage-wise parity: every launch of a block against the exact oracle of THAT launch.

A block stores the result of each einsum (rounded to its storage type) before the next einsum reads
it.  These checkers run the block once through the C ABI with the stage tap open, so that every
tensor a launch read and wrote is available afterwards, and then, launch by launch, evaluate
oracle/stages.py in fp64 on the inputs the GPU launch actually read and compare with what it wrote:
"bf16 in, fp32 accumulate, within 1e-2" (1e-4 for fp32) with no chain of roundings to excuse, and
with the relu mask being the GPU's own h (no ambiguous decisions).  Because each stage's oracle input
is the buffer the previous GPU stage produced in the same run, the composition of the block is
checked too: a launch that read the wrong buffer fails its stage.

At small sizes every output element of every stage is compared.  At full sizes the comparison runs
on sampled rows / columns / (batch, head) pairs that always contain the first and last index of every
slice along every split dimension; every sampled output is summed over the FULL reduction range.
"""
from __future__ import annotations

import numpy as np

from helpers import TOL, Guarded, from_torch, parity_error, to_torch


def _nt(names, a):
    from oracle import NT
    a = np.asarray(a, dtype=np.float64)
    return NT(list(zip(names, a.shape)), a)


def _idx(ix):
    import torch
    return torch.as_tensor(np.asarray(ix, dtype=np.int64), device="cuda")


class Tap:
    """Opens the stage tap on a device buffer; after close(), ``get(name, shape, dtype)`` views the
    k-th tensor tapped under that name."""

    def __init__(self, mtf, nbytes, guard):
        self.mtf = mtf
        self.buf = guard.empty([max(int(nbytes), 256)], "u8")
        mtf.mtf_stage_tap_begin(self.buf)
        self.entries = None

    def close(self):
        n = self.mtf.mtf_stage_tap_end()
        self.entries = [self.mtf.mtf_stage_tap_entry(i) for i in range(n)]
        return self

    def has(self, name):
        return any(n == name for n, _, _ in self.entries)

    def get(self, name, shape, dtype, k=0):
        import torch
        tdt = {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]
        hits = [(o, b) for n, o, b in self.entries if n == name]
        assert len(hits) > k, f"stage tap has no entry {name!r} #{k}: {[e[0] for e in self.entries]}"
        off, nbytes = hits[k]
        n = int(np.prod(shape))
        assert nbytes == n * (2 if dtype == "bf16" else 4), (name, nbytes, shape)
        return self.buf[off:off + nbytes].view(tdt).view(*shape)


class StageReport:
    """Collects the parity metric of every stage and asserts the tolerance at the end."""

    def __init__(self, tol, what):
        self.tol, self.what, self.errs = tol, what, {}

    def add(self, stage, got, ref, tol=None):
        got = np.asarray(got, dtype=np.float64)
        assert np.isfinite(got).all(), f"{self.what}: stage {stage} has non-finite values"
        e = parity_error(got, ref)
        self.errs[stage] = max(self.errs.get(stage, 0.0), e)
        self.tol_of = getattr(self, "tol_of", {})
        self.tol_of[stage] = self.tol if tol is None else tol

    def finish(self):
        bad = {k: e for k, e in self.errs.items() if not e <= self.tol_of[k]}
        assert not bad, f"{self.what}: stages above tolerance {bad} (all: {self.errs})"
        return self.errs


# ---------------------------------------------------------------------------------------------------
# feed-forward block
# ---------------------------------------------------------------------------------------------------

def ffn_stage_checks(rep, T, tok, hid, prefix="", y_residual=None, dx_residual=None):
    """T: dict of device tensors (2-D views, tokens x features): x, dy, w, v, bias (or None), h, y, dhp,
    dx, dw, dv, dbias (or None).  tok / hid: sampled token rows / hidden units (index arrays)."""
    from oracle import stages
    ti, hi = _idx(tok), _idx(hid)
    G = from_torch
    w, v = G(T["w"]), G(T["v"])
    bias = _nt(["f"], G(T["bias"])) if T.get("bias") is not None else None
    W, V = _nt(["d", "f"], w), _nt(["f", "d"], v)
    x_t, dy_t, h_t, dhp_t = G(T["x"][ti]), G(T["dy"][ti]), G(T["h"][ti]), G(T["dhp"][ti])
    # h = relu(x . w + bias)                                    rows of sampled tokens, all hidden units
    ref, _ = stages.contraction(_nt(["t", "d"], x_t), W, ["t", "f"], bias=bias, relu=True)
    rep.add(prefix + "h", h_t, ref.a)
    # y = h . v (+ residual)                                     reads the GPU's stored h
    res = _nt(["t", "d"], G(y_residual[ti])) if y_residual is not None else None
    ref, _ = stages.contraction(_nt(["t", "f"], h_t), V, ["t", "d"], residual=res)
    rep.add(prefix + "y", G(T["y"][ti]), ref.a)
    # dhp = (dy . v^T) * [h > 0]                                 the mask is the GPU's own h
    ref, _ = stages.contraction(_nt(["t", "d"], dy_t), V, ["t", "f"], relu_mask=_nt(["t", "f"], h_t))
    rep.add(prefix + "dhp", dhp_t, ref.a)
    # dx = dhp . w^T (+ residual)                                reads the GPU's stored dhp
    res = _nt(["t", "d"], G(dx_residual[ti])) if dx_residual is not None else None
    ref, _ = stages.contraction(_nt(["t", "f"], dhp_t), W, ["t", "d"], residual=res)
    rep.add(prefix + "dx", G(T["dx"][ti]), ref.a)
    # parameter gradients of sampled hidden units: sums over ALL tokens
    x_all, dy_all = G(T["x"]), G(T["dy"])
    h_c, dhp_c = G(T["h"][:, hi]), G(T["dhp"][:, hi])
    ref, _ = stages.contraction(_nt(["t", "f"], h_c), _nt(["t", "d"], dy_all), ["f", "d"])
    rep.add(prefix + "dv", G(T["dv"][hi, :]), ref.a)
    ref, _ = stages.contraction(_nt(["t", "d"], x_all), _nt(["t", "f"], dhp_c), ["d", "f"])
    rep.add(prefix + "dw", G(T["dw"][:, hi]), ref.a)
    if T.get("dbias") is not None:
        # the column sum is taken from the unrounded values of the dhp launch (it rides in that launch)
        _, pre = stages.contraction(_nt(["t", "d"], dy_all), _nt(["f", "d"], v[np.asarray(hid)]), ["t", "f"], relu_mask=_nt(["t", "f"], h_c))
        rep.add(prefix + "dbias", G(T["dbias"][hi]), stages.reduce_sum(pre, ["f"]).a)


def run_ffn_stagewise(mtf, layout, inp, act_dtype, grad_dtype="f32", tok=None, hid=None, what="ffn"):
    """Forward + backward of the feed-forward block through the C ABI with the stage tap open, then the
    stage checks.  inp: helpers.ffn_inputs(...).  Returns (stage errors, dict of device outputs)."""
    import torch
    dev = {k: to_torch(s) for k, (_, s) in inp.items()}
    N = {k: mtf.named(dev[k], [n for n, _ in d]) for k, (d, _) in inp.items()}
    xd, wd, vd = inp["x"][0], inp["w"][0], inp["v"][0]
    hd = xd[:-1] + [wd[1]]
    D, F = wd[0][1], wd[1][1]
    tshape = [s for _, s in xd[:-1]]
    Tn = int(np.prod(tshape))
    guard = Guarded()
    _alloc = guard.empty
    out = {"h": _alloc(tshape + [F], act_dtype), "y": _alloc(tshape + [D], act_dtype), "dx": _alloc(tshape + [D], act_dtype),
           "dw": _alloc([D, F], grad_dtype), "dv": _alloc([F, D], grad_dtype)}
    if "bias" in inp:
        out["dbias"] = _alloc([F], grad_dtype)
    nm = lambda t, d: mtf.named(t, [n for n, _ in d])
    ws = _alloc([mtf.mtf_ffn_workspace_bytes(layout, N["x"], N["w"])], "u8")
    tap = Tap(mtf, Tn * F * 4 + 4096, guard)
    mtf.mtf_ffn_forward(layout, N["x"], N["w"], N.get("bias"), N["v"], nm(out["h"], hd), nm(out["y"], xd), ws)
    mtf.mtf_ffn_backward(layout, N["x"], N["w"], N["v"], nm(out["h"], hd), N["dy"], nm(out["dx"], xd), nm(out["dw"], wd),
                         nm(out["dbias"], [wd[1]]) if "bias" in inp else None, nm(out["dv"], vd), ws)
    tap.close()
    mtf.mtf_device_status()
    guard.check()
    for k, t in out.items():
        assert bool(torch.isfinite(t).all()), f"{what}: {k} has unwritten or non-finite elements"
    dhp = tap.get("dhp", [Tn, F], act_dtype)
    T = {"x": dev["x"].view(Tn, D), "dy": dev["dy"].view(Tn, D), "w": dev["w"], "v": dev["v"], "bias": dev.get("bias"),
         "h": out["h"].view(Tn, F), "y": out["y"].view(Tn, D), "dhp": dhp, "dx": out["dx"].view(Tn, D), "dw": out["dw"], "dv": out["dv"],
         "dbias": out.get("dbias")}
    rep = StageReport(TOL[act_dtype], what)
    ffn_stage_checks(rep, T, np.arange(Tn) if tok is None else tok, np.arange(F) if hid is None else hid)
    return rep.finish(), out


# ---------------------------------------------------------------------------------------------------
# attention block
# ---------------------------------------------------------------------------------------------------

def attention_stage_checks(rep, T, causal, tok, pairs, wcols, prefix="", y_residual=None, dx_residual=None):
    """T: device tensors in their natural shapes: x, dy [B,L,D]; wq, wk, wv [D,H,K]; wo [H,K,D];
    q, kk, vv, o, do, dq, dkk, dvv [B,L,H,K]; P, dlogits [B,H,L,L]; y, dx [B,L,D]; dwq, dwk, dwv, dwo.
    tok: sampled flat token indices (b * L + l); pairs: sampled (b, h); wcols: sampled (h, k)."""
    from oracle import stages
    G = from_torch
    B, L, D = T["x"].shape
    H, K = T["wq"].shape[1], T["wq"].shape[2]
    s = float(K) ** -0.5
    ti = _idx(tok)
    flat = lambda t: t.reshape(B * L, *t.shape[2:])
    wq, wk, wv = (_nt(["d", "h", "k"], G(T[n])) for n in ("wq", "wk", "wv"))
    wo = _nt(["h", "k", "d"], G(T["wo"]))
    x_t = _nt(["t", "d"], G(flat(T["x"])[ti]))
    dy_t = _nt(["t", "d"], G(flat(T["dy"])[ti]))
    # projections of sampled tokens (all heads)
    for name, wmat in (("q", wq), ("kk", wk), ("vv", wv)):
        ref, _ = stages.contraction(x_t, wmat, ["t", "h", "k"])
        rep.add(prefix + name, G(flat(T[name])[ti]), ref.a)
    # output projection (+ residual) and its input gradient
    res = _nt(["t", "d"], G(flat(y_residual)[ti])) if y_residual is not None else None
    ref, _ = stages.contraction(_nt(["t", "h", "k"], G(flat(T["o"])[ti])), wo, ["t", "d"], residual=res)
    rep.add(prefix + "y", G(flat(T["y"])[ti]), ref.a)
    ref, _ = stages.contraction(dy_t, wo, ["t", "h", "k"])
    rep.add(prefix + "do", G(flat(T["do"])[ti]), ref.a)
    # dx = dq . wq + dkk . wk + dvv . wv (+ residual): one accumulator on the GPU
    terms = [stages.contraction(_nt(["t", "h", "k"], G(flat(T[g])[ti])), wm, ["t", "d"])[0].a for g, wm in (("dq", wq), ("dkk", wk), ("dvv", wv))]
    ref = terms[0] + terms[1] + terms[2]
    if dx_residual is not None:
        ref = ref + G(flat(dx_residual)[ti])
    rep.add(prefix + "dx", G(flat(T["dx"])[ti]), ref)
    # the attention core of sampled (batch, head) pairs: whole rows, all positions
    pos = np.arange(L) if causal else None
    for b, h in pairs:
        q, kk, vv = (_nt(["l", "k"], G(T["q"][b, :, h])), _nt(["m", "k"], G(T["kk"][b, :, h])), _nt(["m", "k"], G(T["vv"][b, :, h])))
        P_g, do_g = G(T["P"][b, h]), G(T["do"][b, :, h])
        lg, _ = stages.contraction(q, kk, ["l", "m"], scale=s)
        rep.add(prefix + "P", P_g, stages.softmax_last(lg, pos).a)
        if causal:
            iu = np.triu_indices(L, 1)
            assert (P_g[iu] == 0.0).all(), "causal weights above the diagonal must be exactly zero"
        Pn = _nt(["l", "m"], P_g)
        ref, _ = stages.contraction(Pn, vv, ["l", "k"])
        rep.add(prefix + "o", G(T["o"][b, :, h]), ref.a)
        don = _nt(["l", "k"], do_g)
        dP, _ = stages.contraction(don, vv, ["l", "m"])
        dlg_ref = stages.softmax_last_backward(Pn, dP).a
        if T.get("dlogits") is not None:
            # the gradient of the logits is a stored stage of its own: the two contractions after it are checked on what was stored
            dlg_g = G(T["dlogits"][b, h])
            rep.add(prefix + "dlogits", dlg_g, dlg_ref)
        else:
            # one launch for the whole backward core: the gradient of the logits never reaches memory, so dq and dkk
            # are held against the exact chain from the launch's own inputs (P, do, vv, q, kk)
            dlg_g = dlg_ref
        ref, _ = stages.contraction(Pn, don, ["m", "k"])
        rep.add(prefix + "dvv", G(T["dvv"][b, :, h]), ref.a)
        dlgn = _nt(["l", "m"], dlg_g)
        ref, _ = stages.contraction(dlgn, kk, ["l", "k"], scale=s)
        rep.add(prefix + "dq", G(T["dq"][b, :, h]), ref.a)
        ref, _ = stages.contraction(dlgn, q, ["m", "k"], scale=s)
        rep.add(prefix + "dkk", G(T["dkk"][b, :, h]), ref.a)
    # parameter gradients of sampled (head, k) columns: sums over ALL tokens
    x_all, dy_all = _nt(["t", "d"], G(flat(T["x"]))), _nt(["t", "d"], G(flat(T["dy"])))
    hs, ks = _idx([h for h, _ in wcols]), _idx([k for _, k in wcols])
    for gname, src in (("dwq", "dq"), ("dwk", "dkk"), ("dwv", "dvv")):
        ref, _ = stages.contraction(x_all, _nt(["t", "c"], G(flat(T[src])[:, hs, ks])), ["d", "c"])
        rep.add(prefix + gname, G(T[gname][:, hs, ks]), ref.a)
    ref, _ = stages.contraction(_nt(["t", "c"], G(flat(T["o"])[:, hs, ks])), dy_all, ["c", "d"])
    rep.add(prefix + "dwo", G(T["dwo"][hs, ks, :]), ref.a)


def _attention_shapes(inp):
    (b, B), (l, L), (d, D) = inp["x"][0]
    (_, _), (h, H), (k, K) = inp["wq"][0]
    v = inp["wv"][0][2][0]
    m = "memory_length"
    return B, L, D, H, K, {"q": [(b, B), (l, L), (h, H), (k, K)], "kk": [(b, B), (m, L), (h, H), (k, K)], "vv": [(b, B), (m, L), (h, H), (v, K)],
                           "P": [(b, B), (h, H), (l, L), (m, L)], "o": [(b, B), (l, L), (h, H), (v, K)]}


def all_samples(B, L, H, K):
    """The sample sets that cover every output element (the default at small sizes)."""
    return np.arange(B * L), [(b, h) for b in range(B) for h in range(H)], [(h, k) for h in range(H) for k in range(K)]


def run_attention_stagewise(mtf, layout, inp, causal, tok=None, pairs=None, wcols=None, what="attention", causal_hint=True):
    """causal_hint: whether the backward call is told that the weights are causal (it is right either way)."""
    import torch
    dev = {k: to_torch(s) for k, (_, s) in inp.items()}
    N = {k: mtf.named(dev[k], [n for n, _ in d]) for k, (d, _) in inp.items()}
    B, L, D, H, K, sd = _attention_shapes(inp)
    sd["y"], sd["dx"] = inp["x"][0], inp["x"][0]
    guard = Guarded()
    _alloc = guard.empty
    out = {n: _alloc([s for _, s in dd], "bf16") for n, dd in sd.items()}
    for n in ("wq", "wk", "wv", "wo"):
        out["d" + n] = _alloc([s for _, s in inp[n][0]], "f32")
        sd["d" + n] = inp[n][0]
    O = {n: mtf.named(t, [x for x, _ in sd[n]]) for n, t in out.items()}
    ws = _alloc([mtf.mtf_attention_workspace_bytes(layout, N["x"], N["wq"], N["wv"])], "u8")
    tap = Tap(mtf, 4 * B * L * H * K * 2 + B * H * L * L * 2 + 8192, guard)
    mtf.mtf_attention_forward(layout, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], causal, None, O["q"], O["kk"], O["vv"], O["P"], O["o"], O["y"], ws)
    mtf.mtf_attention_backward(layout, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], O["q"], O["kk"], O["vv"], O["P"], O["o"], N["dy"], None,
                               O["dx"], O["dwq"], O["dwk"], O["dwv"], O["dwo"], ws, causal=causal and causal_hint)
    tap.close()
    mtf.mtf_device_status()
    guard.check()
    for k, t in out.items():
        assert bool(torch.isfinite(t).all()), f"{what}: {k} has unwritten or non-finite elements"
    T = dict(dev)
    T.update(out)
    for n in ("do", "dq", "dkk", "dvv"):
        T[n] = tap.get(n, [B, L, H, K], "bf16")
    T["dlogits"] = tap.get("dlogits", [B, H, L, L], "bf16") if tap.has("dlogits") else None
    a_tok, a_pairs, a_wcols = all_samples(B, L, H, K)
    rep = StageReport(TOL["bf16"], what)
    attention_stage_checks(rep, T, causal, a_tok if tok is None else tok, a_pairs if pairs is None else pairs, a_wcols if wcols is None else wcols)
    return rep.finish(), out


# ---------------------------------------------------------------------------------------------------
# decoder layer
# ---------------------------------------------------------------------------------------------------

PARAMS = ["wq", "wk", "wv", "wo", "ln1_gamma", "ln1_beta", "w", "bias", "v", "ln2_gamma", "ln2_beta"]
GRAD_FIELD = {"wq": "dwq", "wk": "dwk", "wv": "dwv", "wo": "dwo", "ln1_gamma": "dln1_gamma", "ln1_beta": "dln1_beta", "w": "dw", "bias": "dbias",
              "v": "dv", "ln2_gamma": "dln2_gamma", "ln2_beta": "dln2_beta"}


def run_decoder_stagewise(mtf, layout, inp, tok=None, pairs=None, wcols=None, hid=None, dcols=None, eps=1e-6, what="decoder", causal_hint=True):
    """inp: test_gpu_attention.decoder_case(...).  Runs the decoder layer forward + backward with the
    stage tap open and checks every launch: the attention stages (residual x riding in the output
    projection), layer norm 1, the feed-forward stages on a (residual a), layer norm 2, and the
    backward pass in reverse with the gradient streams ds2, da, ds1 taken from the tap."""
    import torch
    from oracle import stages
    G = from_torch
    dev = {k: to_torch(s) for k, (_, s) in inp.items()}
    N = {k: mtf.named(dev[k], [n for n, _ in d]) for k, (d, _) in inp.items()}
    B, L, D, H, K, sd = _attention_shapes(inp)
    sd["weights"] = sd.pop("P")
    F = inp["w"][0][1][1]
    act = inp["x"][0]
    (b, _), (l, _), _ = act
    sd.update({"s1": act, "a": act, "s2": act, "h": [act[0], act[1], ("d_ff", F)]})
    guard = Guarded()
    _alloc = guard.empty
    saved_t = {n: _alloc([s for _, s in dd], "bf16") for n, dd in sd.items()}
    saved = {n: mtf.named(t, [x for x, _ in sd[n]]) for n, t in saved_t.items()}
    for n in ("stats1", "stats2"):
        saved_t[n] = _alloc([B, L, 2], "f32")
        saved[n] = mtf.named(saved_t[n], [b, l, "stat"])
    params = {k: N[k] for k in PARAMS}
    names = [n for n, _ in act]
    out, dx = _alloc([B, L, D], "bf16"), _alloc([B, L, D], "bf16")
    grads_t = {k: _alloc([s for _, s in inp[k][0]], "f32") for k in PARAMS}
    grads = {GRAD_FIELD[k]: mtf.named(t, [n for n, _ in inp[k][0]]) for k, t in grads_t.items()}
    ws = _alloc([mtf.mtf_decoder_layer_workspace_bytes(layout, N["x"], params)], "u8")
    tap = Tap(mtf, (7 * B * L * D + 2 * B * L * F + B * H * L * L) * 2 + 16384, guard)
    mtf.mtf_decoder_layer_forward(layout, N["x"], params, True, eps, saved, mtf.named(out, names), ws)
    mtf.mtf_decoder_layer_backward(layout, N["x"], params, saved, N["dout"], mtf.named(dx, names), grads, ws, causal=causal_hint)
    tap.close()
    mtf.mtf_device_status()
    guard.check()
    for k, t in list(saved_t.items()) + list(grads_t.items()) + [("out", out), ("dx", dx)]:
        assert bool(torch.isfinite(t).all()), f"{what}: {k} has unwritten or non-finite elements"
    Tn = B * L
    a_tok, a_pairs, a_wcols = all_samples(B, L, H, K)
    tok = a_tok if tok is None else tok
    pairs = a_pairs if pairs is None else pairs
    wcols = a_wcols if wcols is None else wcols
    hid = np.arange(F) if hid is None else hid
    dcols = np.arange(D) if dcols is None else dcols
    ti, ci = _idx(tok), _idx(dcols)
    rep = StageReport(TOL["bf16"], what)
    ds2, da, ds1 = (tap.get(n, [B, L, D], "bf16") for n in ("ds2", "da", "ds1"))
    f2 = lambda t: t.reshape(Tn, t.shape[-1])
    g1, b1, g2, b2 = (_nt(["d"], G(dev[n])) for n in ("ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta"))
    # ---- forward: s1 = x + Attention(x); a = LN1(s1); s2 = a + FFN(a); out = LN2(s2) ----
    A = {"x": dev["x"], "dy": ds1, "wq": dev["wq"], "wk": dev["wk"], "wv": dev["wv"], "wo": dev["wo"], "q": saved_t["q"], "kk": saved_t["kk"],
         "vv": saved_t["vv"], "P": saved_t["weights"], "o": saved_t["o"], "y": saved_t["s1"], "dx": dx, "dwq": grads_t["wq"], "dwk": grads_t["wk"],
         "dwv": grads_t["wv"], "dwo": grads_t["wo"], "dlogits": tap.get("dlogits", [B, H, L, L], "bf16") if tap.has("dlogits") else None}
    for n in ("do", "dq", "dkk", "dvv"):
        A[n] = tap.get(n, [B, L, H, K], "bf16")
    attention_stage_checks(rep, A, True, tok, pairs, wcols, prefix="att.", y_residual=dev["x"], dx_residual=ds1)
    for tag, src, dst, gam, bet, stats in (("ln1", "s1", "a", g1, b1, "stats1"), ("ln2", "s2", None, g2, b2, "stats2")):
        rows = _nt(["t", "d"], G(f2(saved_t[src])[ti]))
        y_ref, mu, r = stages.layernorm_rows(rows, gam, bet, eps)
        rep.add(tag + ".y", G(f2(saved_t[dst] if dst else out)[ti]), y_ref.a)
        st = G(saved_t[stats].reshape(Tn, 2)[ti])
        rep.add(tag + ".mean", st[:, 0], mu, tol=1e-4)
        rep.add(tag + ".rstd", st[:, 1], r, tol=1e-4)
    Ff = {"x": f2(saved_t["a"]), "dy": f2(ds2), "w": dev["w"], "v": dev["v"], "bias": dev["bias"], "h": f2(saved_t["h"]), "y": f2(saved_t["s2"]),
          "dhp": tap.get("dhp", [Tn, F], "bf16"), "dx": f2(da), "dw": grads_t["w"], "dv": grads_t["v"], "dbias": grads_t["bias"]}
    ffn_stage_checks(rep, Ff, tok, hid, prefix="ffn.", y_residual=f2(saved_t["a"]), dx_residual=f2(ds2))
    # ---- backward of the two layer norms: rows of the gradient stream, sampled columns of the parameter gradients ----
    for tag, src, dyt, dxt, gam, gg, gb in (("ln2", "s2", dev["dout"], ds2, g2, "ln2_gamma", "ln2_beta"), ("ln1", "s1", da, ds1, g1, "ln1_gamma", "ln1_beta")):
        ref = stages.layernorm_backward_rows(_nt(["t", "d"], G(f2(saved_t[src])[ti])), _nt(["t", "d"], G(f2(dyt)[ti])), gam, eps)
        rep.add(tag + ".dx", G(f2(dxt)[ti]), ref.a)
        dg, db = stages.layernorm_param_grads(_nt(["t", "d"], G(f2(saved_t[src]))), _nt(["t", "d"], G(f2(dyt))), eps, np.asarray(dcols))
        rep.add(tag + ".dgamma", G(grads_t[gg][ci]), dg)
        rep.add(tag + ".dbeta", G(grads_t[gb][ci]), db)
    res = {"out": out, "dx": dx}
    res.update({"d_" + k: t for k, t in grads_t.items()})
    return rep.finish(), res
