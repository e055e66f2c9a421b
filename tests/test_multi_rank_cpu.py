"""The N > 1 path on CPU: two gloo ranks, each owning one block of the batch (the batch-splitting
mesh dimension mapped onto ranks), run the feed-forward backward pass on their shard and sum the
parameter gradients with the helper the bench uses.  The result must equal the un-split computation
(Algorithm 1 / Section 8.1).  The per-rank arithmetic here is the oracle's: no GPU is involved."""
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


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import NT, DenseOps, blocks
    from paper_1811_02084_b200 import multi_gpu
    B, L, D, F = 4, 6, 8, 16
    ops = DenseOps()
    x = si.normal(3, "x", [B, L, D], "f32").f64
    dy = si.normal(3, "dy", [B, L, D], "f32").f64
    w = NT([("d_model", D), ("d_ff", F)], si.normal(3, "w", [D, F], "f32", D ** -0.5).f64)
    v = NT([("d_ff", F), ("d_model", D)], si.normal(3, "v", [F, D], "f32", F ** -0.5).f64)
    bias = NT([("d_ff", F)], si.normal(3, "bias", [F], "f32", 0.1).f64)
    b0, b1 = multi_gpu.rank_block(B, world, rank)
    dims = [("batch", b1 - b0), ("length", L), ("d_model", D)]
    xs, dys = NT(dims, x[b0:b1]), NT(dims, dy[b0:b1])
    f = blocks.ffn_forward(ops, xs, w, bias, v)
    g = blocks.ffn_backward(ops, xs, w, v, f["h"], dys)
    grads = [torch.from_numpy(g[k].a.copy()) for k in ("dw", "dv", "dbias")]
    # dw and dv through the non-blocking path the bench uses between its launches, dbias through the blocking one
    sync = multi_gpu.GradientSync(dist)
    sync.start(grads[1])
    sync.start(grads[0])
    sync.finish()
    assert sync.pending == []
    multi_gpu.allreduce_gradients(dist, grads[2:])
    slowest = multi_gpu.max_over_ranks(dist, float(rank + 1))
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), dw=grads[0].numpy(), dv=grads[1].numpy(), dbias=grads[2].numpy(),
             dx=g["dx"].a, y=f["y"].a, slowest=slowest, block=np.array([b0, b1]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_batch_split_matches_unsplit(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from oracle import NT, DenseOps, blocks
    B, L, D, F = 4, 6, 8, 16
    ops = DenseOps()
    dims = [("batch", B), ("length", L), ("d_model", D)]
    x, dy = NT(dims, si.normal(3, "x", [B, L, D], "f32").f64), NT(dims, si.normal(3, "dy", [B, L, D], "f32").f64)
    w = NT([("d_model", D), ("d_ff", F)], si.normal(3, "w", [D, F], "f32", D ** -0.5).f64)
    v = NT([("d_ff", F), ("d_model", D)], si.normal(3, "v", [F, D], "f32", F ** -0.5).f64)
    bias = NT([("d_ff", F)], si.normal(3, "bias", [F], "f32", 0.1).f64)
    f = blocks.ffn_forward(ops, x, w, bias, v)
    g = blocks.ffn_backward(ops, x, w, v, f["h"], dy)
    r = [np.load(os.path.join(str(tmp_path), f"rank{i}.npz")) for i in range(world)]
    for k in ("dw", "dv", "dbias"):
        for i in range(world):
            np.testing.assert_allclose(r[i][k], g[k].a, rtol=1e-12, atol=1e-13)          # every rank ends with the sum
    assert [tuple(r[i]["block"]) for i in range(world)] == [(0, 2), (2, 4)]
    np.testing.assert_allclose(np.concatenate([r[0]["dx"], r[1]["dx"]]), g["dx"].a, rtol=1e-12, atol=1e-13)   # activations stay sharded
    np.testing.assert_allclose(np.concatenate([r[0]["y"], r[1]["y"]]), f["y"].a, rtol=1e-12, atol=1e-13)
    assert float(r[0]["slowest"]) == float(r[1]["slowest"]) == 2.0


def test_rank_block_rules():
    from paper_1811_02084_b200 import multi_gpu
    assert [multi_gpu.rank_block(32, 8, r) for r in (0, 3, 7)] == [(0, 4), (12, 16), (28, 32)]
    with pytest.raises(ValueError):
        multi_gpu.rank_block(30, 8, 0)
    multi_gpu.allreduce_gradients(None, [torch.ones(2)])          # single process: no-op
    one = multi_gpu.GradientSync(None)
    one.start(torch.ones(2))
    one.finish()
    assert multi_gpu.max_over_ranks(None, 3.5) == 3.5
