"""Thin ctypes binding of include/mtf.h.  Argument marshalling only: every step of the path runs
inside libmtf_b200.so.  Function names are those of the C ABI.

Tensors are described by ``Named`` objects: dimension names + sizes + dtype (+ a device pointer
taken from a contiguous torch tensor).  Planning-only calls accept descriptors without data.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_uint32, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
_BASE_LIB = os.path.join(_HERE, "libmtf_b200.so")
_SHARE_LIB = os.path.join(_HERE, "libmtf_b200_mc.so")     # optional single-GPU build whose CTA clusters share operand tiles


def _single_gpu_process() -> bool:
    """True only when this process can drive exactly one GPU and no multi-rank launcher started it."""
    for var in ("WORLD_SIZE", "LOCAL_WORLD_SIZE", "OMPI_COMM_WORLD_SIZE", "PMI_SIZE", "SLURM_NTASKS"):
        try:
            if int(os.environ.get(var, "1")) > 1:
                return False
        except ValueError:
            return False
    try:
        import torch
        return torch.cuda.device_count() == 1
    except Exception:
        return False


def _choose_library() -> str:
    """libmtf_b200.so always, unless MTF_CLUSTER_SHARE=1 asks for the single-GPU build AND that
    library exists AND this is a single-GPU, single-rank process."""
    if os.environ.get("MTF_CLUSTER_SHARE") == "1" and os.path.exists(_SHARE_LIB) and _single_gpu_process():
        return _SHARE_LIB
    return _BASE_LIB


LIB_PATH = _choose_library()

MTF_F32, MTF_BF16 = 0, 1
MTF_KERNEL_SIMT, MTF_KERNEL_TCGEN05 = 0, 1
MTF_REDUCE_NONE, MTF_REDUCE_CHAINED, MTF_REDUCE_WORKSPACE = 0, 1, 2
STATUS_NAMES = ["MTF_OK", "MTF_ERR_INVALID_ARG", "MTF_ERR_DUPLICATE_DIM", "MTF_ERR_UNKNOWN_DIM",
                "MTF_ERR_SIZE_MISMATCH", "MTF_ERR_ILLEGAL_LAYOUT", "MTF_ERR_NOT_DIVISIBLE", "MTF_ERR_UNSUPPORTED",
                "MTF_ERR_WORKSPACE_TOO_SMALL", "MTF_ERR_CUDA", "MTF_ERR_TIMEOUT"]


class mtf_dim(Structure):
    _fields_ = [("name", c_char_p), ("size", c_int64)]


class mtf_tensor(Structure):
    _fields_ = [("data", c_void_p), ("dtype", c_int), ("ndim", c_int32), ("dims", POINTER(mtf_dim))]


class mtf_epilogue(Structure):
    _fields_ = [("scale", c_float), ("relu", c_int32), ("bias", POINTER(mtf_tensor)),
                ("relu_mask", POINTER(mtf_tensor)), ("residual", POINTER(mtf_tensor)),
                ("reduce_sum_out", POINTER(mtf_tensor))]


class mtf_decoder_params(Structure):
    _fields_ = [(n, POINTER(mtf_tensor)) for n in ("wq", "wk", "wv", "wo", "ln1_gamma", "ln1_beta", "w", "bias", "v", "ln2_gamma", "ln2_beta")]


class mtf_decoder_saved(Structure):
    _fields_ = [(n, POINTER(mtf_tensor)) for n in ("q", "kk", "vv", "weights", "o", "s1", "stats1", "a", "h", "s2", "stats2")]


class mtf_decoder_grads(Structure):
    _fields_ = [(n, POINTER(mtf_tensor)) for n in ("dwq", "dwk", "dwv", "dwo", "dln1_gamma", "dln1_beta", "dw", "dbias", "dv", "dln2_gamma", "dln2_beta")]


RANK_ALLREDUCE_FN = ctypes.CFUNCTYPE(c_int, c_void_p, c_void_p, c_int64, c_int, c_void_p)     # (user, data, count, dtype, stream) -> status
RANK_WAIT_FN = ctypes.CFUNCTYPE(c_int, c_void_p, c_void_p)                                    # (user, stream) -> status


class mtf_update_params(Structure):
    _fields_ = [("lr", c_float), ("momentum", c_float), ("weight_decay", c_float)]


MTF_RESHAPE_NONE, MTF_RESHAPE_ALLGATHER, MTF_RESHAPE_SLICE, MTF_RESHAPE_ALLTOALL = 0, 1, 2, 3


class MtfError(RuntimeError):
    def __init__(self, status: int, message: str):
        self.status = status
        self.code = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else f"MTF_ERR_{status}"
        super().__init__(f"{self.code}: {message}")


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: the CUDA library has not been built. Build it with "
            "`python paper_1811_02084_b200/build.py` (needs nvcc; there is no CPU fallback).")
    L = ctypes.CDLL(LIB_PATH)
    vp = c_void_p
    sig = {
        "mtf_mesh_create": [c_int32, POINTER(mtf_dim), POINTER(vp)],
        "mtf_mesh_destroy": [vp],
        "mtf_mesh_size": [vp, POINTER(c_int64)],
        "mtf_mesh_coords": [vp, c_int64, POINTER(c_int64)],
        "mtf_layout": [vp, c_int32, POINTER(c_char_p), POINTER(c_char_p), POINTER(vp)],
        "mtf_layout_destroy": [vp],
        "mtf_layout_check_tensor": [vp, c_int32, POINTER(mtf_dim)],
        "mtf_slice_map": [vp, c_int32, POINTER(mtf_dim), c_int64, POINTER(c_int64), POINTER(c_int64)],
        "mtf_slice_gather": [vp, POINTER(mtf_tensor), c_int64, vp, vp],
        "mtf_einsum_plan": [vp, c_int32, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_epilogue), POINTER(vp)],
        "mtf_plan_destroy": [vp],
        "mtf_plan_workspace_bytes": [vp, POINTER(c_size_t)],
        "mtf_plan_cost": [vp, POINTER(c_int64), POINTER(c_int64), POINTER(c_int64), POINTER(c_int32)],
        "mtf_plan_info": [vp, POINTER(c_int32), POINTER(c_int32), POINTER(c_int64), POINTER(c_int64), POINTER(c_uint32)],
        "mtf_einsum_exec": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_epilogue), vp, c_size_t, vp],
        "mtf_einsum": [vp, c_char_p, c_int32, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_epilogue), vp, c_size_t, vp],
        "mtf_einsum_builtin_scratch": [vp, c_char_p, c_int32, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_epilogue), vp],
        "mtf_einsum_workspace_bytes": [vp, c_int32, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_epilogue), POINTER(c_size_t)],
        "mtf_plan_force": [c_int32, c_int32],
        "mtf_hint_independent": [],
        "mtf_ffn_forward": [vp] + [POINTER(mtf_tensor)] * 6 + [vp, c_size_t, vp],
        "mtf_ffn_backward": [vp] + [POINTER(mtf_tensor)] * 9 + [vp, c_size_t, vp],
        "mtf_ffn_workspace_bytes": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(c_size_t)],
        "mtf_reduce_sum": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_softmax_forward": [vp, POINTER(mtf_tensor), c_int32, POINTER(mtf_tensor), vp],
        "mtf_softmax_backward": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_einsum_softmax": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), c_float, c_int32, POINTER(mtf_tensor), vp, c_size_t, vp],
        "mtf_einsum_softmax_backward": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), vp, c_size_t, vp],
        "mtf_layernorm_forward": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), c_float, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_layernorm_backward": [vp] + [POINTER(mtf_tensor)] * 8 + [vp, c_size_t, vp],
        "mtf_layernorm_workspace_bytes": [c_int64, POINTER(c_size_t)],
        "mtf_attention_forward": [vp] + [POINTER(mtf_tensor)] * 5 + [c_int32] + [POINTER(mtf_tensor)] * 7 + [vp, c_size_t, vp],
        "mtf_attention_backward": [vp] + [POINTER(mtf_tensor)] * 5 + [c_int32] + [POINTER(mtf_tensor)] * 12 + [vp, c_size_t, vp],
        "mtf_attention_workspace_bytes": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(c_size_t)],
        "mtf_decoder_layer_forward": [vp, POINTER(mtf_tensor), POINTER(mtf_decoder_params), c_int32, c_float, POINTER(mtf_decoder_saved), POINTER(mtf_tensor), vp, c_size_t, vp],
        "mtf_decoder_layer_backward": [vp, POINTER(mtf_tensor), POINTER(mtf_decoder_params), c_int32, POINTER(mtf_decoder_saved), POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_decoder_grads), vp, c_size_t, vp],
        "mtf_decoder_layer_workspace_bytes": [vp, POINTER(mtf_tensor), POINTER(mtf_decoder_params), POINTER(c_size_t)],
        "mtf_device_status": [POINTER(c_int32)],
        "mtf_layout_bind_ranks": [vp, c_char_p, c_int32, c_int32, RANK_ALLREDUCE_FN, RANK_WAIT_FN, vp, POINTER(vp)],
        "mtf_rank_box": [vp, c_int32, POINTER(mtf_dim), POINTER(c_int64), POINTER(c_int64)],
        "mtf_plan_needs_rank_sum": [vp, POINTER(c_int32)],
        "mtf_rank_wait": [vp, vp],
        "mtf_update": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_update_params), vp],
        "mtf_reshape_plan": [vp, c_int32, POINTER(mtf_dim), POINTER(c_char_p), POINTER(c_int32), POINTER(c_int64)],
        "mtf_transpose": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_slice_scatter": [vp, vp, c_int64, POINTER(mtf_tensor), vp],
        "mtf_layout_search": [vp, c_int32, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), c_int32, POINTER(c_char_p), ctypes.c_double,
                              POINTER(c_int32), POINTER(ctypes.c_double), POINTER(c_int64)],
        "mtf_embedding_forward": [vp, vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_embedding_backward": [vp, vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_softmax_xent_forward": [vp, POINTER(mtf_tensor), vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_softmax_xent_backward": [vp, POINTER(mtf_tensor), vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp],
        "mtf_xent_forward": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), vp, c_size_t, vp],
        "mtf_xent_backward": [vp, POINTER(mtf_tensor), POINTER(mtf_tensor), vp, POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor), POINTER(mtf_tensor),
                              POINTER(mtf_tensor), vp, c_size_t, vp],
        "mtf_debug_wait_test": [c_int64, c_int32],
        "mtf_stage_tap_begin": [vp, c_size_t],
        "mtf_stage_tap_end": [POINTER(c_int32)],
        "mtf_stage_tap_entry": [c_int32, POINTER(c_char_p), POINTER(c_size_t), POINTER(c_size_t)],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = c_int
    L.mtf_status_string.argtypes = [c_int]
    L.mtf_status_string.restype = c_char_p
    L.mtf_last_error.argtypes = []
    L.mtf_last_error.restype = c_char_p
    L.mtf_launch_count.argtypes = []
    L.mtf_launch_count.restype = c_int64
    return L


_lib = _load()


def _check(status: int):
    if status != 0:
        raise MtfError(status, _lib.mtf_last_error().decode("utf-8", "replace"))


def _dims_array(dims):
    arr = (mtf_dim * max(len(dims), 1))()
    keep = []
    for i, (n, s) in enumerate(dims):
        b = n.encode("utf-8")
        keep.append(b)
        arr[i].name = b
        arr[i].size = int(s)
    return arr, keep


def _dtype_code(dtype) -> int:
    if dtype in (MTF_F32, "f32", "float32"):
        return MTF_F32
    if dtype in (MTF_BF16, "bf16", "bfloat16"):
        return MTF_BF16
    name = str(dtype)
    if name == "torch.float32":
        return MTF_F32
    if name == "torch.bfloat16":
        return MTF_BF16
    raise MtfError(1, f"unsupported dtype {dtype!r}")


class Named:
    """A named tensor view: ``dims`` = [(name, size), ...] in storage order, dtype code, device pointer."""

    def __init__(self, dims, dtype, data_ptr=None, owner=None):
        self.dims = [(str(n), int(s)) for n, s in dims]
        self.dtype = _dtype_code(dtype)
        self.ptr = data_ptr
        self.owner = owner            # keeps the torch tensor alive
        self._dims_arr, self._keep = _dims_array(self.dims)
        self.c = mtf_tensor(c_void_p(data_ptr) if data_ptr else None, self.dtype, len(self.dims), self._dims_arr)

    @property
    def names(self):
        return [n for n, _ in self.dims]


def named(t, names) -> Named:
    """Describe a contiguous torch tensor (any device; the pointer is passed as is) with dim names."""
    if len(names) != t.dim():
        raise MtfError(1, f"{len(names)} names for a {t.dim()}-d tensor")
    if not t.is_contiguous():
        raise MtfError(1, "tensors must be dense row-major (contiguous)")
    return Named(list(zip(names, t.shape)), t.dtype, t.data_ptr(), owner=t)


def desc(dims, dtype) -> Named:
    """A descriptor without data (for planning calls)."""
    return Named(dims, dtype)


def _stream(stream):
    if stream is not None:
        return c_void_p(int(stream))
    try:
        import torch
        if torch.cuda.is_available():
            return c_void_p(torch.cuda.current_stream().cuda_stream)
    except Exception:
        pass
    return c_void_p(0)


def _ws(workspace):
    if workspace is None:
        return c_void_p(0), 0
    return c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size()


class Epilogue:
    def __init__(self, scale=1.0, relu=False, bias: Named | None = None, relu_mask: Named | None = None,
                 residual: Named | None = None, reduce_sum_out: Named | None = None):
        self.refs = (bias, relu_mask, residual, reduce_sum_out)
        self.c = mtf_epilogue(float(scale), 1 if relu else 0,
                              ctypes.pointer(bias.c) if bias is not None else None,
                              ctypes.pointer(relu_mask.c) if relu_mask is not None else None,
                              ctypes.pointer(residual.c) if residual is not None else None,
                              ctypes.pointer(reduce_sum_out.c) if reduce_sum_out is not None else None)


def _epi(e):
    return byref(e.c) if e is not None else None


class Mesh:
    def __init__(self, handle, dims):
        self.handle = handle
        self.dims = dims

    def __del__(self):
        if getattr(self, "handle", None):
            _lib.mtf_mesh_destroy(self.handle)
            self.handle = None


class Layout:
    def __init__(self, handle, mesh_dims, rules):
        self.handle = handle
        self.mesh_dims = mesh_dims
        self.rules = rules

    def __del__(self):
        if getattr(self, "handle", None):
            _lib.mtf_layout_destroy(self.handle)
            self.handle = None


class Plan:
    def __init__(self, handle):
        self.handle = handle

    def __del__(self):
        if getattr(self, "handle", None):
            _lib.mtf_plan_destroy(self.handle)
            self.handle = None


# ---- the C ABI, name for name ---------------------------------------------------------------------

def mtf_mesh_create(mesh_dims) -> Mesh:
    arr, _keep = _dims_array(mesh_dims)
    h = c_void_p()
    _check(_lib.mtf_mesh_create(len(mesh_dims), arr, byref(h)))
    return Mesh(h, list(mesh_dims))


def mtf_mesh_size(mesh: Mesh) -> int:
    n = c_int64()
    _check(_lib.mtf_mesh_size(mesh.handle, byref(n)))
    return n.value


def mtf_mesh_coords(mesh: Mesh, processor: int):
    out = (c_int64 * len(mesh.dims))()
    _check(_lib.mtf_mesh_coords(mesh.handle, processor, out))
    return list(out)


def mtf_layout(mesh: Mesh, rules) -> Layout:
    n = len(rules)
    t = (c_char_p * max(n, 1))(*[r[0].encode() for r in rules])
    m = (c_char_p * max(n, 1))(*[r[1].encode() for r in rules])
    h = c_void_p()
    _check(_lib.mtf_layout(mesh.handle, n, t, m, byref(h)))
    return Layout(h, list(mesh.dims), list(rules))


def mtf_layout_bind_ranks(layout: Layout, mesh_dim: str, world: int, rank: int, collective=None) -> Layout:
    """This rank's part of ``layout`` when mesh dimension ``mesh_dim`` is spread over ``world`` ranks.
    ``collective``: an object with ctypes callbacks ``start_cb`` (RANK_ALLREDUCE_FN) and ``wait_cb``
    (RANK_WAIT_FN), e.g. multi_gpu.RankCollective; None = the caller sums the flagged outputs itself."""
    h = c_void_p()
    start = collective.start_cb if collective is not None else RANK_ALLREDUCE_FN()
    wait = collective.wait_cb if collective is not None else RANK_WAIT_FN()
    _check(_lib.mtf_layout_bind_ranks(layout.handle, mesh_dim.encode(), int(world), int(rank), start, wait, None, byref(h)))
    mesh_dims = [(n, s // world if n == mesh_dim else s) for n, s in layout.mesh_dims]
    out = Layout(h, mesh_dims, list(layout.rules))
    out.collective = collective          # keeps the callbacks alive as long as the handle
    return out


def mtf_rank_box(bound_layout: Layout, global_dims):
    arr, _keep = _dims_array(global_dims)
    offs = (c_int64 * max(len(global_dims), 1))()
    sizes = (c_int64 * max(len(global_dims), 1))()
    _check(_lib.mtf_rank_box(bound_layout.handle, len(global_dims), arr, offs, sizes))
    return list(offs)[:len(global_dims)], list(sizes)[:len(global_dims)]


def mtf_plan_needs_rank_sum(plan: Plan) -> int:
    f = c_int32()
    _check(_lib.mtf_plan_needs_rank_sum(plan.handle, byref(f)))
    return f.value


def mtf_rank_wait(bound_layout: Layout, stream=None) -> None:
    _check(_lib.mtf_rank_wait(bound_layout.handle, _stream(stream)))


def mtf_layout_check_tensor(layout: Layout, dims) -> None:
    arr, _keep = _dims_array(dims)
    _check(_lib.mtf_layout_check_tensor(layout.handle, len(dims), arr))


def mtf_slice_map(layout: Layout, dims, processor: int):
    arr, _keep = _dims_array(dims)
    offs = (c_int64 * max(len(dims), 1))()
    sizes = (c_int64 * max(len(dims), 1))()
    _check(_lib.mtf_slice_map(layout.handle, len(dims), arr, processor, offs, sizes))
    return list(offs)[:len(dims)], list(sizes)[:len(dims)]


def mtf_slice_gather(layout: Layout, glob: Named, processor: int, out_slice, stream=None) -> None:
    _check(_lib.mtf_slice_gather(layout.handle, byref(glob.c), processor, c_void_p(out_slice.data_ptr()), _stream(stream)))


def _tensor_array(ts):
    arr = (mtf_tensor * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = t.c
    return arr


def mtf_einsum_plan(layout: Layout, ins, out: Named, epilogue: Epilogue | None = None) -> Plan:
    h = c_void_p()
    _check(_lib.mtf_einsum_plan(layout.handle, len(ins), _tensor_array(ins), byref(out.c), _epi(epilogue), byref(h)))
    return Plan(h)


def mtf_plan_workspace_bytes(plan: Plan) -> int:
    b = c_size_t()
    _check(_lib.mtf_plan_workspace_bytes(plan.handle, byref(b)))
    return b.value


def mtf_plan_cost(plan: Plan) -> dict:
    a, b, c, d = c_int64(), c_int64(), c_int64(), c_int32()
    _check(_lib.mtf_plan_cost(plan.handle, byref(a), byref(b), byref(c), byref(d)))
    return {"macs_per_proc": a.value, "allreduce_values": b.value, "slice_elems": c.value, "n_reduce_mesh_dims": d.value}


def mtf_plan_info(plan: Plan) -> dict:
    k, r, n, g, m = c_int32(), c_int32(), c_int64(), c_int64(), c_uint32()
    _check(_lib.mtf_plan_info(plan.handle, byref(k), byref(r), byref(n), byref(g), byref(m)))
    return {"kernel_kind": k.value, "reduce_mode": r.value, "n_slices": n.value, "group_size": g.value,
            "reduce_mesh_dim_mask": m.value}


def mtf_einsum_exec(plan: Plan, ins, out: Named, epilogue: Epilogue | None = None, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_einsum_exec(plan.handle, _tensor_array(ins), byref(out.c), _epi(epilogue), wp, wb, _stream(stream)))


def mtf_einsum(layout: Layout, equation, ins, out: Named, epilogue: Epilogue | None = None, workspace=None,
               stream=None) -> None:
    wp, wb = _ws(workspace)
    eq = equation.encode() if equation is not None else None
    _check(_lib.mtf_einsum(layout.handle, eq, len(ins), _tensor_array(ins), byref(out.c), _epi(epilogue), wp, wb,
                           _stream(stream)))


def mtf_einsum_builtin_scratch(layout: Layout, equation, ins, out: Named, epilogue: Epilogue | None = None, stream=None) -> None:
    """mtf_einsum without a workspace argument, for callers that cannot allocate device memory: the
    partial tiles of a workspace-mode group sum go to a fixed 32 MiB array inside the library."""
    eq = equation.encode() if equation is not None else None
    _check(_lib.mtf_einsum_builtin_scratch(layout.handle, eq, len(ins), _tensor_array(ins), byref(out.c), _epi(epilogue),
                                           _stream(stream)))


def mtf_einsum_workspace_bytes(layout: Layout, ins, out: Named, epilogue: Epilogue | None = None) -> int:
    b = c_size_t()
    _check(_lib.mtf_einsum_workspace_bytes(layout.handle, len(ins), _tensor_array(ins), byref(out.c), _epi(epilogue), byref(b)))
    return b.value


def mtf_hint_independent() -> None:
    """The next contraction of this thread is independent of the launch before it on its stream (see mtf.h)."""
    _check(_lib.mtf_hint_independent())


def mtf_plan_force(kernel_kind: int = -1, reduce_mode: int = -1) -> None:
    _check(_lib.mtf_plan_force(kernel_kind, reduce_mode))


def _p(t: Named | None):
    return byref(t.c) if t is not None else None


def mtf_ffn_forward(layout, x, w, bias, v, h_saved, y, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_ffn_forward(layout.handle, _p(x), _p(w), _p(bias), _p(v), _p(h_saved), _p(y), wp, wb, _stream(stream)))


def mtf_ffn_backward(layout, x, w, v, h_saved, dy, dx, dw, dbias, dv, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_ffn_backward(layout.handle, _p(x), _p(w), _p(v), _p(h_saved), _p(dy), _p(dx), _p(dw), _p(dbias),
                                 _p(dv), wp, wb, _stream(stream)))


def mtf_ffn_workspace_bytes(layout, x, w) -> int:
    b = c_size_t()
    _check(_lib.mtf_ffn_workspace_bytes(layout.handle, _p(x), _p(w), byref(b)))
    return b.value


def mtf_reduce_sum(layout, inp: Named, out: Named, stream=None) -> None:
    _check(_lib.mtf_reduce_sum(layout.handle, _p(inp), _p(out), _stream(stream)))


def mtf_softmax_forward(layout, logits: Named, causal: bool, weights: Named, stream=None) -> None:
    _check(_lib.mtf_softmax_forward(layout.handle, _p(logits), 1 if causal else 0, _p(weights), _stream(stream)))


def mtf_softmax_backward(layout, weights: Named, dweights: Named, dlogits: Named, stream=None) -> None:
    _check(_lib.mtf_softmax_backward(layout.handle, _p(weights), _p(dweights), _p(dlogits), _stream(stream)))


def mtf_einsum_softmax(layout, a: Named, b: Named, scale: float, causal: bool, weights: Named, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_einsum_softmax(layout.handle, _p(a), _p(b), float(scale), 1 if causal else 0, _p(weights), wp, wb, _stream(stream)))


def mtf_einsum_softmax_backward(layout, a: Named, b: Named, weights: Named, dlogits: Named, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_einsum_softmax_backward(layout.handle, _p(a), _p(b), _p(weights), _p(dlogits), wp, wb, _stream(stream)))


def mtf_layernorm_forward(layout, x, gamma, beta, eps, y, stats, stream=None) -> None:
    _check(_lib.mtf_layernorm_forward(layout.handle, _p(x), _p(gamma), _p(beta), float(eps), _p(y), _p(stats), _stream(stream)))


def mtf_layernorm_backward(layout, dy, x, stats, gamma, residual, dx, dgamma, dbeta, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_layernorm_backward(layout.handle, _p(dy), _p(x), _p(stats), _p(gamma), _p(residual), _p(dx), _p(dgamma), _p(dbeta),
                                       wp, wb, _stream(stream)))


def mtf_layernorm_workspace_bytes(row_length: int) -> int:
    b = c_size_t()
    _check(_lib.mtf_layernorm_workspace_bytes(int(row_length), byref(b)))
    return b.value


def mtf_attention_forward(layout, x, wq, wk, wv, wo, causal, residual, q, kk, vv, weights, o, y, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_attention_forward(layout.handle, _p(x), _p(wq), _p(wk), _p(wv), _p(wo), 1 if causal else 0, _p(residual), _p(q), _p(kk),
                                      _p(vv), _p(weights), _p(o), _p(y), wp, wb, _stream(stream)))


def mtf_attention_backward(layout, x, wq, wk, wv, wo, q, kk, vv, weights, o, dy, dx_residual, dx, dwq, dwk, dwv, dwo, workspace=None,
                           stream=None, causal=False) -> None:
    """causal: a hint (True promises that `weights` came from a causal forward call; False is always right)."""
    wp, wb = _ws(workspace)
    _check(_lib.mtf_attention_backward(layout.handle, _p(x), _p(wq), _p(wk), _p(wv), _p(wo), 1 if causal else 0, _p(q), _p(kk), _p(vv), _p(weights), _p(o), _p(dy),
                                       _p(dx_residual), _p(dx), _p(dwq), _p(dwk), _p(dwv), _p(dwo), wp, wb, _stream(stream)))


def mtf_attention_workspace_bytes(layout, x, wq, wv) -> int:
    b = c_size_t()
    _check(_lib.mtf_attention_workspace_bytes(layout.handle, _p(x), _p(wq), _p(wv), byref(b)))
    return b.value


def _struct_of(cls, tensors: dict):
    s = cls()
    for name, _t in cls._fields_:
        t = tensors.get(name)
        setattr(s, name, ctypes.pointer(t.c) if t is not None else None)
    return s


def mtf_decoder_layer_forward(layout, x, params: dict, causal, eps, saved: dict, out, workspace=None, stream=None) -> None:
    """params / saved: dicts of Named keyed by the field names of mtf_decoder_params / mtf_decoder_saved."""
    wp, wb = _ws(workspace)
    ps, sv = _struct_of(mtf_decoder_params, params), _struct_of(mtf_decoder_saved, saved)
    _check(_lib.mtf_decoder_layer_forward(layout.handle, _p(x), byref(ps), 1 if causal else 0, float(eps), byref(sv), _p(out), wp, wb,
                                          _stream(stream)))


def mtf_decoder_layer_backward(layout, x, params: dict, saved: dict, dout, dx, grads: dict, workspace=None, stream=None, causal=False) -> None:
    wp, wb = _ws(workspace)
    ps, sv, gs = _struct_of(mtf_decoder_params, params), _struct_of(mtf_decoder_saved, saved), _struct_of(mtf_decoder_grads, grads)
    _check(_lib.mtf_decoder_layer_backward(layout.handle, _p(x), byref(ps), 1 if causal else 0, byref(sv), _p(dout), _p(dx), byref(gs), wp, wb, _stream(stream)))


def mtf_decoder_layer_workspace_bytes(layout, x, params: dict) -> int:
    b = c_size_t()
    ps = _struct_of(mtf_decoder_params, params)
    _check(_lib.mtf_decoder_layer_workspace_bytes(layout.handle, _p(x), byref(ps), byref(b)))
    return b.value


def mtf_update(layout, grad: Named, master: Named, momentum: Named | None, param: Named | None, lr: float, momentum_coef: float = 0.0,
               weight_decay: float = 0.0, stream=None) -> None:
    hp = mtf_update_params(float(lr), float(momentum_coef), float(weight_decay))
    _check(_lib.mtf_update(layout.handle, _p(grad), _p(master), _p(momentum), _p(param), byref(hp), _stream(stream)))


def mtf_reshape_plan(layout: Layout, in_dims, out_names):
    """Per mesh dimension: (pattern code, elements one processor would receive)."""
    arr, _keep = _dims_array(in_dims)
    names = (c_char_p * max(len(out_names), 1))(*[n.encode() for n in out_names])
    r = len(layout.mesh_dims)
    pat, rec = (c_int32 * r)(), (c_int64 * r)()
    _check(_lib.mtf_reshape_plan(layout.handle, len(in_dims), arr, names, pat, rec))
    return list(pat), list(rec)


def mtf_transpose(layout, inp: Named, out: Named, stream=None) -> None:
    _check(_lib.mtf_transpose(layout.handle, _p(inp), _p(out), _stream(stream)))


def mtf_slice_scatter(layout: Layout, slice_tensor, processor: int, glob: Named, stream=None) -> None:
    _check(_lib.mtf_slice_scatter(layout.handle, c_void_p(slice_tensor.data_ptr()), processor, byref(glob.c), _stream(stream)))


def mtf_layout_search(mesh: Mesh, einsums, names, comm_weight: float):
    """einsums: [(in0, in1, out)] of descriptors.  Returns (rules, cost, footprint) of the cheapest legal layout."""
    a0, a1, ao = _tensor_array([e[0] for e in einsums]), _tensor_array([e[1] for e in einsums]), _tensor_array([e[2] for e in einsums])
    nm = (c_char_p * max(len(names), 1))(*[n.encode() for n in names])
    chosen = (c_int32 * max(len(names), 1))()
    cost, foot = ctypes.c_double(), c_int64()
    _check(_lib.mtf_layout_search(mesh.handle, len(einsums), a0, a1, ao, len(names), nm, float(comm_weight), chosen, byref(cost), byref(foot)))
    rules = [(n, mesh.dims[chosen[i]][0]) for i, n in enumerate(names) if chosen[i] >= 0]
    return rules, cost.value, foot.value


def mtf_embedding_forward(layout, ids, table: Named, x: Named, stream=None) -> None:
    """ids: contiguous int32 device tensor, one id per token."""
    _check(_lib.mtf_embedding_forward(layout.handle, c_void_p(ids.data_ptr()), _p(table), _p(x), _stream(stream)))


def mtf_embedding_backward(layout, ids, dx: Named, dtable: Named, stream=None) -> None:
    _check(_lib.mtf_embedding_backward(layout.handle, c_void_p(ids.data_ptr()), _p(dx), _p(dtable), _stream(stream)))


def mtf_softmax_xent_forward(layout, logits: Named, targets, lse: Named, loss: Named, stream=None) -> None:
    _check(_lib.mtf_softmax_xent_forward(layout.handle, _p(logits), c_void_p(targets.data_ptr()), _p(lse), _p(loss), _stream(stream)))


def mtf_softmax_xent_backward(layout, logits: Named, targets, lse: Named, dloss: Named, stream=None) -> None:
    _check(_lib.mtf_softmax_xent_backward(layout.handle, _p(logits), c_void_p(targets.data_ptr()), _p(lse), _p(dloss), _stream(stream)))


def mtf_xent_forward(layout, h: Named, wout: Named, targets, logits: Named, lse: Named, loss: Named, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_xent_forward(layout.handle, _p(h), _p(wout), c_void_p(targets.data_ptr()), _p(logits), _p(lse), _p(loss), wp, wb, _stream(stream)))


def mtf_xent_backward(layout, h: Named, wout: Named, targets, logits: Named, lse: Named, dloss: Named, dh: Named, dwout: Named, workspace=None,
                      stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_lib.mtf_xent_backward(layout.handle, _p(h), _p(wout), c_void_p(targets.data_ptr()), _p(logits), _p(lse), _p(dloss), _p(dh), _p(dwout), wp, wb,
                                  _stream(stream)))


def mtf_status_string(status: int) -> str:
    return _lib.mtf_status_string(status).decode()


def mtf_last_error() -> str:
    return _lib.mtf_last_error().decode("utf-8", "replace")


def mtf_device_status() -> int:
    """Synchronises the device; raises MtfError(MTF_ERR_TIMEOUT) when a bounded wait gave up."""
    c = c_int32()
    _check(_lib.mtf_device_status(byref(c)))
    return c.value


def mtf_stage_tap_begin(buffer) -> None:
    """Open the stage tap on a device byte buffer (a contiguous torch tensor)."""
    _check(_lib.mtf_stage_tap_begin(c_void_p(buffer.data_ptr()), buffer.numel() * buffer.element_size()))


def mtf_stage_tap_end() -> int:
    n = c_int32()
    _check(_lib.mtf_stage_tap_end(byref(n)))
    return n.value


def mtf_stage_tap_entry(index: int):
    """(name, byte offset, byte size) of one tapped intermediate."""
    name, off, size = c_char_p(), c_size_t(), c_size_t()
    _check(_lib.mtf_stage_tap_entry(index, byref(name), byref(off), byref(size)))
    return name.value.decode(), off.value, size.value


def mtf_debug_wait_test(limit_cycles: int = 0, withhold_one_signal: bool = False) -> None:
    """Testing hook: see mtf_debug_wait_test in include/mtf.h."""
    _check(_lib.mtf_debug_wait_test(int(limit_cycles), 1 if withhold_one_signal else 0))


def mtf_launch_count() -> int:
    return int(_lib.mtf_launch_count())
