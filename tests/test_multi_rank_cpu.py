"""The N > 1 path on CPU: two gloo ranks drive the library's own multi-rank host logic through the
C ABI - mtf_layout_bind_ranks, mtf_rank_box, the plans' "needs a sum across ranks" flags and the
collective hooks the binding provides over torch.distributed - for both ways the path shards:
a batch split (Algorithm 1 / Section 8.1: the parameter gradients are summed) and a split of the
hidden dimension (Section 8.2: y and dx are summed).  What the library says is checked against the
oracle's lowering on a mesh whose first dimension is the ranks: the rank's box of every tensor is
the union of its processors' slices, and an einsum needs a sum across ranks exactly when the oracle's
Allreduce for it runs over that mesh dimension.  No GPU is involved (planning and hooks are host code)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import seeded_inputs as si


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


B, L, D, F, H, K = 4, 6, 8, 16, 4, 8
MESH = [("ranks", 2), ("cols", 2)]
SPLITS = {"batch over ranks": [("batch", "ranks"), ("d_ff", "cols"), ("heads", "cols")],
          "model dims over ranks": [("d_ff", "ranks"), ("heads", "ranks"), ("batch", "cols")]}
ACT, HID = [("batch", B), ("length", L), ("d_model", D)], [("batch", B), ("length", L), ("d_ff", F)]
W, V = [("d_model", D), ("d_ff", F)], [("d_ff", F), ("d_model", D)]
Q = [("batch", B), ("length", L), ("heads", H), ("d_k", K)]
WQ, WO = [("d_model", D), ("heads", H), ("d_k", K)], [("heads", H), ("d_k", K), ("d_model", D)]
# (name, input dims, output dims): the einsums of the feed-forward block and the attention projections
EINSUMS = [("h", [ACT, W], HID), ("y", [HID, V], ACT), ("dhp", [ACT, V], HID), ("dv", [HID, ACT], V), ("dw", [ACT, HID], W), ("dx", [HID, W], ACT),
           ("q", [ACT, WQ], Q), ("att_y", [Q, WO], ACT), ("dwq", [ACT, Q], WQ), ("dwo", [Q, ACT], WO), ("att_dx", [Q, WQ], ACT)]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_1811_02084_b200 as mtf
    from paper_1811_02084_b200 import multi_gpu
    from oracle import NT, Layout, LoweredOps, Mesh
    coll = multi_gpu.RankCollective(dist, device="cpu")
    for split, rules in SPLITS.items():
        lay = mtf.mtf_layout(mtf.mtf_mesh_create(MESH), rules)
        bound = mtf.mtf_layout_bind_ranks(lay, "ranks", world, rank, coll)
        olay = Layout(Mesh(MESH), rules)
        mine = [p for p in range(olay.mesh.P) if olay.mesh.coords(p)[0] == rank]
        local = {}
        # the rank's box of every tensor = the union of its processors' slices
        for dims in (ACT, HID, W, V, Q, WQ, WO):
            offs, sizes = mtf.mtf_rank_box(bound, dims)
            lo = [min(olay.slice_box(dims, p)[0][i] for p in mine) for i in range(len(dims))]
            hi = [max(olay.slice_box(dims, p)[0][i] + olay.slice_box(dims, p)[1][i] for p in mine) for i in range(len(dims))]
            assert offs == lo and [o + s for o, s in zip(offs, sizes)] == hi, (split, dims, offs, sizes, lo, hi)
            local[tuple(dims)] = [(n, s) for (n, _), s in zip(dims, sizes)]
        # an einsum needs a sum across ranks exactly when the oracle's Allreduce runs over mesh dimension 0
        for name, ins, out in EINSUMS:
            ops = LoweredOps(olay)
            ops.einsum([ops.lower(NT(d, si.small_integers(1, name + str(i), [s for _, s in d]))) for i, d in enumerate(ins)], [n for n, _ in out])
            want = any(0 in over for _tag, over, _n in ops.allreduce_log)
            plan = mtf.mtf_einsum_plan(bound, [mtf.desc(local[tuple(d)], "bf16") for d in ins], mtf.desc(local[tuple(out)], "f32"))
            assert bool(mtf.mtf_plan_needs_rank_sum(plan) & 1) == want, (split, name, want)
            # and, inside the rank, the group sum runs over the remaining mesh dimension exactly as the oracle's does
            info = mtf.mtf_plan_info(plan)
            want_local = any(1 in over for _tag, over, _n in ops.allreduce_log)
            assert (info["group_size"] > 1) == want_local, (split, name)
        # non-linear stages cannot ride in a launch whose result is a partial sum across ranks
        if split == "model dims over ranks":
            bias = mtf.desc([("d_model", D)], "f32")
            with pytest.raises(mtf.MtfError) as e:
                mtf.mtf_einsum_plan(bound, [mtf.desc(local[tuple(HID)], "bf16"), mtf.desc(local[tuple(V)], "bf16")], mtf.desc(local[tuple(ACT)], "f32"),
                                    mtf.Epilogue(bias=bias, relu=True))
            assert e.value.code == "MTF_ERR_UNSUPPORTED"
    # the hooks over gloo: start is non-blocking, wait completes them; f32 and bf16 buffers
    a = np.full(1000, float(rank + 1), dtype=np.float32)
    b = (np.arange(64, dtype=np.float32) * (rank + 1))
    bb = si.round_to_bf16_bits(b)
    assert coll.start_cb(None, a.ctypes.data, a.size, mtf.MTF_F32, None) == 0
    assert coll.start_cb(None, bb.ctypes.data, bb.size, mtf.MTF_BF16, None) == 0
    assert len(coll.pending) == 2
    assert coll.wait_cb(None, None) == 0 and coll.pending == [] and coll.error is None
    assert np.all(a == sum(range(1, world + 1)))
    assert np.array_equal(si.bf16_bits_to_f64(bb), np.arange(64) * float(sum(range(1, world + 1))))
    slowest = multi_gpu.max_over_ranks(dist, float(rank + 1))
    assert slowest == float(world)
    open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_library_host_path_matches_oracle_lowering(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(os.path.join(str(tmp_path), f"ok{r}")) for r in range(world))


def test_bind_ranks_argument_checks():
    import paper_1811_02084_b200 as mtf
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("rows", 4), ("cols", 3)]), [("batch", "rows")])
    for args, code in ((("nope", 2, 0), "MTF_ERR_UNKNOWN_DIM"), (("cols", 2, 0), "MTF_ERR_NOT_DIVISIBLE"), (("rows", 2, 2), "MTF_ERR_INVALID_ARG")):
        with pytest.raises(mtf.MtfError) as e:
            mtf.mtf_layout_bind_ranks(lay, *args)
        assert e.value.code == code
    one = mtf.mtf_layout_bind_ranks(lay, "rows", 1, 0)          # world 1 changes nothing
    plan = mtf.mtf_einsum_plan(one, [mtf.desc([("batch", 8), ("k", 16)], "bf16"), mtf.desc([("k", 16), ("n", 8)], "bf16")], mtf.desc([("batch", 8), ("n", 8)], "f32"))
    assert mtf.mtf_plan_needs_rank_sum(plan) == 0
    bound = mtf.mtf_layout_bind_ranks(lay, "rows", 2, 1)
    with pytest.raises(mtf.MtfError):
        mtf.mtf_layout_bind_ranks(bound, "cols", 3, 0)            # one rank-spanning mesh dimension
    # the fused reduce_sum over a batch split across ranks is a partial sum too (bit 1)
    x, v = mtf.desc([("batch", 4), ("d", 16)], "bf16"), mtf.desc([("f", 8), ("d", 16)], "bf16")
    plan = mtf.mtf_einsum_plan(bound, [x, v], mtf.desc([("batch", 4), ("f", 8)], "bf16"),
                               mtf.Epilogue(relu_mask=mtf.desc([("batch", 4), ("f", 8)], "bf16"), reduce_sum_out=mtf.desc([("f", 8)], "f32")))
    assert mtf.mtf_plan_needs_rank_sum(plan) == 2
