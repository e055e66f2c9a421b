#!/usr/bin/env python
"""Benchmark of the hot path: Transformer feed-forward block, forward + backward, as layout-lowered
named-dimension einsums on one B200 (or N replicas of the batch-split mesh dimension on N GPUs).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--layout mp8|dp8|none|mp16] [--split dp|mp] [--impl reference]

One step = mtf_ffn_forward + mtf_ffn_backward through the C ABI on the workload
tokens 8192 (batch 32 x length 256), d_model 1024, d_ff 8192, bf16 storage / fp32 accumulation
(six tensor-core contractions, 12 * tokens * d_model * d_ff flop).  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = {"batch": 32, "length": 256, "d_model": 1024, "d_ff": 8192}
LAYOUTS = {
    "none": ([("all", 1)], []),
    "dp8": ([("all", 8)], [("batch", "all")]),
    "mp8": ([("all", 8)], [("d_ff", "all")]),
    "mp16": ([("all", 16)], [("d_ff", "all")]),
    # Section 8.3: the two-dimensional layout (batch over rows, hidden over columns) and the three-dimensional one
    # (additionally the input / output dimension over planes: every matrix tiled over two mesh dimensions)
    "2d": ([("rows", 2), ("cols", 4)], [("batch", "rows"), ("d_ff", "cols")]),
    "3d": ([("rows", 2), ("cols", 2), ("planes", 2)], [("batch", "rows"), ("d_ff", "cols"), ("d_model", "planes")]),
}
# dram__bytes_read.sum + dram__bytes_write.sum per contraction launch, averaged over the six launches of a
# step of this workload (one ncu capture; the summary under profiles/ names the command and the commit)
NCU_DRAM_BYTES_PER_LAUNCH = 167.9e6
NCU_TRAFFIC_COMMIT = "abd89d6"
METRIC = "transformer_ffn_fwd_bwd_tflops"
UNIT = "TFLOP/s"


def ffn_flops(tokens, d_model, d_ff):
    return 12.0 * tokens * d_model * d_ff


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"bf16_sustained": float(d["bf16_tflops_sustained"]), "bf16_burst": float(d["bf16_tflops"]),
                    "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
        except Exception:
            pass
    return {"bf16_sustained": 1400.0, "bf16_burst": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs (read only)."""

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None
            return self
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def _run(self):
        nv = self._nvml
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80, "sw_power_cap": 0x4}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=1.0)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------------

def oracle_step_fn(tokens: int, seed: int = 0):
    import seeded_inputs as si
    from oracle import NT, DenseOps, blocks
    d_model, d_ff = WORKLOAD["d_model"], WORKLOAD["d_ff"]
    ops = DenseOps()
    x = NT([("batch", 1), ("length", tokens), ("d_model", d_model)], si.normal(seed, "x", [1, tokens, d_model], "bf16").f64)
    dy = NT(x.dims, si.normal(seed, "dy", [1, tokens, d_model], "bf16").f64)
    w = NT([("d_model", d_model), ("d_ff", d_ff)], si.normal(seed, "w", [d_model, d_ff], "bf16", d_model ** -0.5).f64)
    v = NT([("d_ff", d_ff), ("d_model", d_model)], si.normal(seed, "v", [d_ff, d_model], "bf16", d_ff ** -0.5).f64)
    bias = NT([("d_ff", d_ff)], si.normal(seed, "bias", [d_ff], "f32", 0.1).f64)

    def step():
        f = blocks.ffn_forward(ops, x, w, bias, v)
        blocks.ffn_backward(ops, x, w, v, f["h"], dy)
    return step


def time_oracle(tokens: int, steps: int, warmup: int):
    step = oracle_step_fn(tokens)
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / max(steps, 1)
    return dt, ffn_flops(tokens, WORKLOAD["d_model"], WORKLOAD["d_ff"]) / dt / 1e12


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    # size the per-step sample so that the whole run takes about two minutes
    dt1, _ = time_oracle(1, 1, 1)
    budget = 120.0 / max(args.steps + args.warmup, 1)
    tokens = int(max(1, min(256, budget / max(dt1, 1e-6))))
    dt, tflops = time_oracle(tokens, args.steps, args.warmup)
    sample = f"ffn fwd+bwd on {tokens} of {WORKLOAD['batch'] * WORKLOAD['length']} tokens (full d_model, d_ff), fp64 loop nest"
    line = {"impl": "reference", "metric": METRIC, "value": tflops, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": "transformer_ffn_fwd_bwd tokens=8192 d_model=1024 d_ff=8192", "sampled_tokens": tokens},
            "cpu_baseline": {"value": tflops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": tflops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------------

def to_device(s):
    """seeded_inputs.Stored -> device tensor with exactly those bytes."""
    import numpy as np
    import torch
    if s.dtype == "bf16":
        return torch.from_numpy(s.bits.view(np.int16)).view(torch.bfloat16).cuda()
    return torch.from_numpy(s.bits).cuda()


def event_time(fn, reps, stream, warmup=3):
    """Average device time of fn() in ms: one CUDA-event pair around `reps` back-to-back calls."""
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def run_ours(args):
    import torch
    import seeded_inputs as si

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1 or os.environ.get("MTF_BENCH_DIST"):      # (the variable: exercise the N > 1 code path with one rank)
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local_rank))
    import paper_1811_02084_b200 as mtf
    from paper_1811_02084_b200 import multi_gpu

    B, L, D, F = WORKLOAD["batch"], WORKLOAD["length"], WORKLOAD["d_model"], WORKLOAD["d_ff"]
    T = B * L
    # Per-GPU work is fixed (weak scaling).  With N ranks one mesh dimension ("gpus") spans them:
    #   --split dp: batch -> gpus   (global batch N x 32; every rank its own tokens; dw, dv, dbias are summed: Algorithm 1 line 2)
    #   --split mp: d_ff  -> gpus   (global d_ff N x 8192; every rank its own hidden units; y and dx are summed: Section 8.2)
    # The other dimension keeps the virtual mesh of --layout inside each rank.
    seed_x = 1000 * rank if args.split == "dp" else 0
    seed_w = 0 if args.split == "dp" else 1000 * rank
    host = {
        "x": si.normal(seed_x, "x", [B, L, D], "bf16"),
        "dy": si.normal(seed_x, "dy", [B, L, D], "bf16"),
        "w": si.normal(seed_w, "w", [D, F], "bf16", D ** -0.5),
        "v": si.normal(seed_w, "v", [F, D], "bf16", F ** -0.5),
        "bias": si.normal(seed_w, "bias", [F], "f32", 0.1),
    }
    t = {k: to_device(s) for k, s in host.items()}
    h = torch.empty(B, L, F, dtype=torch.bfloat16, device="cuda")
    y = torch.empty(B, L, D, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty_like(y)
    dw = torch.empty(D, F, dtype=torch.float32, device="cuda")
    dv = torch.empty(F, D, dtype=torch.float32, device="cuda")
    dbias = torch.empty(F, dtype=torch.float32, device="cuda")
    act, wn, vn, hn = ["batch", "length", "d_model"], ["d_model", "d_ff"], ["d_ff", "d_model"], ["batch", "length", "d_ff"]
    N = {"x": mtf.named(t["x"], act), "dy": mtf.named(t["dy"], act), "w": mtf.named(t["w"], wn), "v": mtf.named(t["v"], vn),
         "bias": mtf.named(t["bias"], ["d_ff"]), "h": mtf.named(h, hn), "y": mtf.named(y, act),
         "dx": mtf.named(dx, act), "dw": mtf.named(dw, wn), "dv": mtf.named(dv, vn), "dbias": mtf.named(dbias, ["d_ff"])}

    collective = multi_gpu.RankCollective(dist) if dist is not None else None
    layouts = {}
    for name, (mesh_dims, rules) in LAYOUTS.items():
        if dist is None:
            layouts[name] = mtf.mtf_layout(mtf.mtf_mesh_create(mesh_dims), rules)
            continue
        # the rank-spanning mesh dimension in front of the virtual mesh; the dimension it takes leaves the inner rules
        taken = "batch" if args.split == "dp" else "d_ff"
        inner = [(td, md) for td, md in rules if td != taken]
        glob = mtf.mtf_layout(mtf.mtf_mesh_create([("gpus", world)] + list(mesh_dims)), [(taken, "gpus")] + inner)
        layouts[name] = mtf.mtf_layout_bind_ranks(glob, "gpus", world, rank, collective)
    ws_bytes = max(mtf.mtf_ffn_workspace_bytes(l, N["x"], N["w"]) for l in layouts.values())
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step(lay, xin=None, dyin=None, yout=None, dxout=None):
        # the sums across ranks are started by the library behind the launch that produces each partial
        # result (hooks of the rank-bound layout) and awaited before the block call returns
        mtf.mtf_ffn_forward(lay, xin or N["x"], N["w"], N["bias"], N["v"], N["h"], yout or N["y"], ws)
        mtf.mtf_ffn_backward(lay, xin or N["x"], N["w"], N["v"], N["h"], dyin or N["dy"], dxout or N["dx"], N["dw"], N["dbias"], N["dv"], ws)

    def timed(lay, steps, warmup, sampler=None):
        for _ in range(warmup):
            step(lay)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = mtf.mtf_launch_count()
        e0.record(stream)
        for _ in range(steps):
            step(lay)
        e1.record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop() if sampler else None
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        launches = mtf.mtf_launch_count() - n0
        ms = multi_gpu.max_over_ranks(dist, ms, "cuda")
        return ms / steps, launches, clocks

    flops_step = ffn_flops(T, D, F)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    ms_step, launches, clocks = timed(layouts[args.layout], args.steps, max(args.warmup, 3), sampler)
    mtf.mtf_device_status()
    if collective is not None and collective.error is not None:
        raise collective.error
    value = world * flops_step / (ms_step * 1e-3) / 1e12

    per_layout = {}
    if world == 1 and not args.main_only:
        for name, lay in layouts.items():
            if name == args.layout:
                per_layout[name] = value
                continue
            ms_l, _, _ = timed(lay, max(args.steps // 2, 5), 3)
            per_layout[name] = flops_step / (ms_l * 1e-3) / 1e12

    if args.main_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms_step, "gpu_launches": launches,
                              "config": {"workload": f"tokens={T} d_model={D} d_ff={F}", "layout": args.layout}, "note": "main-only run"}), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return
    # end to end: the step's inputs come from pinned host memory and its results go back, every step.
    # Three streams (copy in, compute, copy out) and two sets of device buffers: step i's inputs are
    # copied while step i-1 computes and step i-2's results return; every step still moves its own
    # 32 MiB in and 32 MiB out inside the timed region.
    hx, hdy = t["x"].cpu().pin_memory(), t["dy"].cpu().pin_memory()
    hy, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
    lay = layouts[args.layout]
    sets = []
    for q in range(2):
        bufs = {"x": torch.empty_like(t["x"]), "dy": torch.empty_like(t["dy"]), "y": torch.empty_like(y), "dx": torch.empty_like(dx)}
        names = {k: mtf.named(v, act) for k, v in bufs.items()}
        sets.append((bufs, names))
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    in_ready = [torch.cuda.Event() for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]
    out_done = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        q = i & 1
        bufs, names = sets[q]
        with torch.cuda.stream(s_in):
            s_in.wait_event(done[q])                    # the step that last read this input set has finished
            bufs["x"].copy_(hx, non_blocking=True)
            bufs["dy"].copy_(hdy, non_blocking=True)
            in_ready[q].record(s_in)
        stream.wait_event(in_ready[q])
        stream.wait_event(out_done[q])                  # the results of the step that last used this output set are on the host
        step(lay, names["x"], names["dy"], names["y"], names["dx"])
        done[q].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(done[q])
            hy.copy_(bufs["y"], non_blocking=True)
            hdx.copy_(bufs["dx"], non_blocking=True)
            out_done[q].record(s_out)

    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    e2e_steps = max(args.steps // 4, 6)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    s_in.wait_event(e0)
    for i in range(e2e_steps):
        e2e_step(i)
    stream.wait_stream(s_out)                           # the last results are on the host before the clock stops
    stream.wait_stream(s_in)
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_ms = multi_gpu.max_over_ranks(dist, e2e_ms, "cuda")
    e2e_value = world * flops_step / (e2e_ms * 1e-3) / 1e12
    act_bytes = hx.numel() * hx.element_size()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # ---- the dominant kernel, launch by launch: the six contractions of a step timed one at a time (CUDA events
    # on the launching stream, 50 back-to-back repeats each), next to torch.matmul on the same shapes
    per_contraction, avg_launch_ms = None, ms_step / 6
    if world == 1:
        dhp = torch.empty(B, L, F, dtype=torch.bfloat16, device="cuda")
        ndhp = mtf.named(dhp, hn)
        calls = {
            "h = relu(x.w + bias)": (lambda: mtf.mtf_einsum(lay, None, [N["x"], N["w"]], N["h"], mtf.Epilogue(relu=True, bias=N["bias"]), workspace=ws), (T, F, D)),
            "y = h.v": (lambda: mtf.mtf_einsum(lay, None, [N["h"], N["v"]], N["y"], None, workspace=ws), (T, D, F)),
            "dhp = (dy.v^T)*[h>0], dbias": (lambda: mtf.mtf_einsum(lay, None, [N["dy"], N["v"]], ndhp, mtf.Epilogue(relu_mask=N["h"], reduce_sum_out=N["dbias"]), workspace=ws), (T, F, D)),
            "dv = h^T.dy": (lambda: mtf.mtf_einsum(lay, None, [N["h"], N["dy"]], N["dv"], None, workspace=ws), (F, D, T)),
            "dw = x^T.dhp": (lambda: mtf.mtf_einsum(lay, None, [N["x"], ndhp], N["dw"], None, workspace=ws), (D, F, T)),
            "dx = dhp.w^T": (lambda: mtf.mtf_einsum(lay, None, [ndhp, N["w"]], N["dx"], None, workspace=ws), (T, D, F)),
        }
        x2, dy2, h2, dhp2 = t["x"].view(T, D), t["dy"].view(T, D), h.view(T, F), dhp.view(T, F)
        o_tf, o_td = torch.empty(T, F, dtype=torch.bfloat16, device="cuda"), torch.empty(T, D, dtype=torch.bfloat16, device="cuda")
        o_fd, o_df = torch.empty(F, D, dtype=torch.bfloat16, device="cuda"), torch.empty(D, F, dtype=torch.bfloat16, device="cuda")
        lib = {
            "h = relu(x.w + bias)": lambda: torch.matmul(x2, t["w"], out=o_tf), "y = h.v": lambda: torch.matmul(h2, t["v"], out=o_td),
            "dhp = (dy.v^T)*[h>0], dbias": lambda: torch.matmul(dy2, t["v"].t(), out=o_tf), "dv = h^T.dy": lambda: torch.matmul(h2.t(), dy2, out=o_fd),
            "dw = x^T.dhp": lambda: torch.matmul(x2.t(), dhp2, out=o_df), "dx = dhp.w^T": lambda: torch.matmul(dhp2, t["w"].t(), out=o_td),
        }
        per_contraction = {}
        for name, (fn, (m_, n_, k_)) in calls.items():
            ms_c = event_time(fn, 50, stream)
            ms_l = event_time(lib[name], 50, stream)
            per_contraction[name] = {"ms": ms_c, "tflops": 2.0 * m_ * n_ * k_ / (ms_c * 1e-3) / 1e12, "torch_matmul_ms": ms_l,
                                     "ratio_to_torch_matmul": ms_c / ms_l, "m_n_k": [m_, n_, k_]}
        avg_launch_ms = sum(c["ms"] for c in per_contraction.values()) / len(per_contraction)
        mtf.mtf_device_status()
    flops_per_launch = flops_step / 6
    achieved = flops_per_launch / (avg_launch_ms * 1e-3) / 1e12

    # which way the sums over a split reduced dimension were realised (Section 6: the Allreduce of the
    # mesh group) in the contractions of this layout that have one, and the workspace they moved
    mode_name = {0: "none", 1: "chained in the accumulator", 2: "fp32 fragments in the workspace"}
    dsc = lambda t_, names: mtf.desc(list(zip(names, t_.shape)), "bf16" if t_.dtype == torch.bfloat16 else "f32")
    group_sums = {}
    for tag, ins, out in (("y", [(h, hn), (t["v"], vn)], (y, act)), ("dx", [(h, hn), (t["w"], wn)], (dx, act)),
                          ("dw", [(t["x"], act), (h, hn)], (dw, wn)), ("dv", [(h, hn), (t["dy"], act)], (dv, vn))):
        plan = mtf.mtf_einsum_plan(lay, [dsc(a_, n_) for a_, n_ in ins], dsc(*out))
        info = mtf.mtf_plan_info(plan)
        if info["group_size"] > 1 or mtf.mtf_plan_needs_rank_sum(plan):
            group_sums[tag] = {"group_size": info["group_size"], "mode": mode_name.get(info["reduce_mode"], str(info["reduce_mode"])),
                               "workspace_bytes": mtf.mtf_plan_workspace_bytes(plan) if info["reduce_mode"] == 2 else 0,
                               "summed_across_ranks": bool(mtf.mtf_plan_needs_rank_sum(plan) & 1)}

    # the same step back to back for two seconds: the rate the GPU settles at under its power limit
    sustained = None
    if world == 1 and not args.no_sustained:
        n_sus = max(int(2000.0 / ms_step), 50)
        ms_sus, _, clocks_sus = timed(lay, n_sus, 3, ClockSampler(physical_gpu_index(local_rank)))
        v_sus = flops_step / (ms_sus * 1e-3) / 1e12
        sustained = {"ms_per_step": ms_sus, "value": v_sus, "unit": UNIT, "steps": n_sus,
                     "sm_mhz": clocks_sus.get("sm_mhz") if clocks_sus else None, "reasons": clocks_sus.get("reasons") if clocks_sus else None,
                     "peak": peaks["bf16_sustained"], "frac": v_sus / peaks["bf16_sustained"], "frac_of_datasheet_2250": v_sus / 2250.0,
                     "note": "whole steps (launch gaps included) against the sustained torch.matmul rate: both seconds long, both under the power cap"}

    # roofline of the dominant kernel: like for like.  A timed region under a second runs at the boost clock and
    # is held against the burst peak (best-of-10 torch.matmul); seconds-long regions against the sustained peak.
    region_s = ms_step * args.steps * 1e-3
    regime = "sustained" if region_s >= 1.0 else "burst"
    traffic = NCU_DRAM_BYTES_PER_LAUNCH if (T, D, F) == (8192, 1024, 8192) else None
    peak = peaks["bf16_sustained"] if regime == "sustained" else peaks["bf16_burst"]
    roofline = {"bound": "tensor", "kernel": "gemm_tcgen05_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": traffic, "traffic_captured_at_commit": NCU_TRAFFIC_COMMIT, "regime": regime,
                "peak_source": f"bf16_tflops{'_sustained' if regime == 'sustained' else ''} of MEASURED_PEAKS.json ({peaks['source']})",
                "frac_of_datasheet_2250": achieved / 2250.0, "flops_per_launch": flops_per_launch, "avg_launch_ms": avg_launch_ms,
                "avg_launch_ms_note": "mean of the six contractions timed one at a time (50 repeats each)" if per_contraction else "step time / 6",
                "step_ms_over_6_launches": ms_step / 6, "per_contraction": per_contraction,
                "sustained_regime": {"achieved": sustained["value"], "peak": peaks["bf16_sustained"], "frac": sustained["frac"]} if sustained else None}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cores = len(os.sched_getaffinity(0))
        tokens = 192
        dt, tf = time_oracle(tokens, 1, 0)
        cpu = {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"ffn fwd+bwd on {tokens} of {T} tokens (full d_model, d_ff), fp64 loop nest, {dt:.1f} s"}

    secondary = None
    if world == 1 and not args.no_secondary:
        del sets, hx, hdy, hy, hdx
        torch.cuda.empty_cache()
        secondary = run_secondary(mtf, peaks)

    multi = "single GPU"
    if world > 1:
        multi = ("batch -> ranks (mesh dimension 'gpus'); dw, dv, dbias summed over ranks with NCCL, each started behind its contraction" if args.split == "dp"
                 else "d_ff -> ranks (mesh dimension 'gpus'); y and dx summed over ranks with NCCL behind their contractions")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"transformer_ffn_fwd_bwd tokens={T} (batch {B} x length {L}) d_model={D} d_ff={F} per GPU",
                       "layout": args.layout, "mesh": LAYOUTS[args.layout][0], "rules": LAYOUTS[args.layout][1],
                       "grad_dtype": "f32", "l2": "inputs larger than L2 (working set ~0.6 GB per step), no flush",
                       "library": os.path.basename(mtf.binding.LIB_PATH), "multi_gpu": multi},
            "clocks": clocks, "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 2 * act_bytes,
                                      "d2h_bytes_per_step": 2 * act_bytes, "ms_per_step": e2e_ms},
            "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu, "per_layout_tflops": per_layout,
            "group_sums": group_sums, "sustained_2s": sustained,
            "frac_of_datasheet_bf16_peak": value / world / 2250.0, "secondary": secondary}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------------
# secondary workloads (records inside the headline line): attention block (config 3), decoder layer (config 5)
# and the memory-bound kernels, on seeded inputs
# ------------------------------------------------------------------------------------------------------

def block_case(seed, dec, B=None):
    """Seeded inputs of config 3 (attention: batch 16, length 512, d_model 1024, 16 heads of 64) or config 5
    (decoder layer: batch 64, length 256, d_model 2048, 32 heads of 64, d_ff 8192): name -> (Stored, dim names)."""
    import seeded_inputs as si
    B0, L, D, H, K, F = (64, 256, 2048, 32, 64, 8192) if dec else (16, 512, 1024, 16, 64, 0)
    B = B or B0
    act = ["batch", "length", "d_model"]
    T = {"x": (si.normal(seed, "x", [B, L, D], "bf16"), act), "dout": (si.normal(seed, "dy", [B, L, D], "bf16"), act),
         "wq": (si.normal(seed, "wq", [D, H, K], "bf16", D ** -0.5), ["d_model", "heads", "d_k"]),
         "wk": (si.normal(seed, "wk", [D, H, K], "bf16", D ** -0.5), ["d_model", "heads", "d_k"]),
         "wv": (si.normal(seed, "wv", [D, H, K], "bf16", D ** -0.5), ["d_model", "heads", "d_v"]),
         "wo": (si.normal(seed, "wo", [H, K, D], "bf16", (H * K) ** -0.5), ["heads", "d_v", "d_model"])}
    if dec:
        T.update({"w": (si.normal(seed, "w", [D, F], "bf16", D ** -0.5), ["d_model", "d_ff"]),
                  "v": (si.normal(seed, "v", [F, D], "bf16", F ** -0.5), ["d_ff", "d_model"]),
                  "bias": (si.normal(seed, "bias", [F], "f32", 0.1), ["d_ff"])})
        for n, shift in (("ln1_gamma", 1.0), ("ln1_beta", 0.0), ("ln2_gamma", 1.0), ("ln2_beta", 0.0)):
            T[n] = (si.normal(seed, n, [D], "f32", 0.1, shift), ["d_model"])
    return T, (B, L, D, H, K, F)


def block_step(mtf, dec, B=None):
    """Builds the step function of the attention block (config 3) or the decoder layer (config 5) on seeded inputs.
    Returns (step, flops per step, description, tensors kept alive)."""
    import torch
    bf, f32 = torch.bfloat16, torch.float32
    host, (B, L, D, H, K, F) = block_case(0, dec, B)
    mesh, rules = ([("rows", 4), ("cols", 8)], [("batch", "rows"), ("heads", "cols"), ("d_ff", "cols")]) if dec else \
                  ([("rows", 4), ("cols", 4)], [("batch", "rows"), ("heads", "cols")])
    lay = mtf.mtf_layout(mtf.mtf_mesh_create(mesh), rules)
    act = ["batch", "length", "d_model"]
    T = {k: (to_device(s), names) for k, (s, names) in host.items()}
    N = {k: mtf.named(t_, names) for k, (t_, names) in T.items()}
    m = "memory_length"
    sd = {"q": ((B, L, H, K), ["batch", "length", "heads", "d_k"]), "kk": ((B, L, H, K), ["batch", m, "heads", "d_k"]),
          "vv": ((B, L, H, K), ["batch", m, "heads", "d_v"]), "weights": ((B, H, L, L), ["batch", "heads", "length", m]),
          "o": ((B, L, H, K), ["batch", "length", "heads", "d_v"]), "s1": ((B, L, D), act), "a": ((B, L, D), act), "s2": ((B, L, D), act)}
    if dec:
        sd["h"] = ((B, L, F), ["batch", "length", "d_ff"])
    keep = {n: torch.empty(shape, dtype=bf, device="cuda") for n, (shape, _) in sd.items()}
    S = {n: mtf.named(keep[n], sd[n][1]) for n in keep}
    for n in ("stats1", "stats2"):
        keep[n] = torch.empty(B, L, 2, dtype=f32, device="cuda")
        S[n] = mtf.named(keep[n], ["batch", "length", "stat"])
    out, dx = torch.empty(B, L, D, dtype=bf, device="cuda"), torch.empty(B, L, D, dtype=bf, device="cuda")
    params = [k for k in T if k not in ("x", "dout")]
    gname = {"wq": "dwq", "wk": "dwk", "wv": "dwv", "wo": "dwo", "ln1_gamma": "dln1_gamma", "ln1_beta": "dln1_beta", "w": "dw", "bias": "dbias",
             "v": "dv", "ln2_gamma": "dln2_gamma", "ln2_beta": "dln2_beta"}
    gt = {k: torch.empty_like(T[k][0], dtype=f32) for k in params}
    G = {gname[k]: mtf.named(gt[k], T[k][1]) for k in params}
    P = {k: N[k] for k in params}
    if dec:
        ws = torch.empty(mtf.mtf_decoder_layer_workspace_bytes(lay, N["x"], P), dtype=torch.uint8, device="cuda")
        flops = 3 * (8.0 * B * L * D * H * K + 4.0 * B * H * L * L * K + 4.0 * B * L * D * F)

        def step():
            mtf.mtf_decoder_layer_forward(lay, N["x"], P, True, 1e-6, S, mtf.named(out, act), ws)
            mtf.mtf_decoder_layer_backward(lay, N["x"], P, S, N["dout"], mtf.named(dx, act), G, ws, causal=True)
    else:
        ws = torch.empty(mtf.mtf_attention_workspace_bytes(lay, N["x"], N["wq"], N["wv"]), dtype=torch.uint8, device="cuda")
        flops = 3 * (8.0 * B * L * D * H * K + 4.0 * B * H * L * L * K)

        def step():
            mtf.mtf_attention_forward(lay, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], False, None, S["q"], S["kk"], S["vv"], S["weights"], S["o"],
                                      mtf.named(out, act), ws)
            mtf.mtf_attention_backward(lay, N["x"], N["wq"], N["wk"], N["wv"], N["wo"], S["q"], S["kk"], S["vv"], S["weights"], S["o"], N["dout"], None,
                                       mtf.named(dx, act), G["dwq"], G["dwk"], G["dwv"], G["dwo"], ws)
    desc = {"workload": ("decoder layer, config 5" if dec else "attention block, config 3") + f": batch={B} length={L} d_model={D} heads={H} d_k={K}" + (f" d_ff={F} causal" if dec else ""),
            "mesh": mesh, "rules": rules, "flops_per_step": flops,
            "flops_note": "dense-equivalent contraction flops (projections, attention core, FFN), 2 per multiply-add, forward + backward = 3x forward"}
    return step, flops, desc, (T, keep, gt, out, dx, ws, lay)


def run_secondary(mtf, peaks, blocks=True, reps=None):
    """Records for the other workloads and for the memory-bound kernels, each timed with CUDA events on seeded inputs.
    blocks=False leaves out the attention block and the decoder layer; reps overrides the repeat counts (profiler captures)."""
    import torch
    import seeded_inputs as si
    stream = torch.cuda.current_stream()
    out = []
    if reps is not None:
        timer = lambda fn, n, st_, warmup=3: event_time(fn, reps, st_, warmup=1)
    else:
        timer = event_time
    for dec in ((False, True) if blocks else ()):
        step, flops, desc, keep = block_step(mtf, dec)
        ms = event_time(step, 20, stream, warmup=3)
        mtf.mtf_device_status()
        tf = flops / (ms * 1e-3) / 1e12
        out.append({"metric": "transformer_" + ("decoder_layer" if dec else "attention") + "_fwd_bwd_tflops", "value": tf, "unit": UNIT, "ms_per_step": ms,
                    "dtype": "bf16", "data": "synthetic (seeded)", "config": desc,
                    "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_burst"], "frac": tf / peaks["bf16_burst"], "unit": "TFLOP/s",
                                 "note": "whole block (contractions + row kernels) against the burst torch.matmul rate; timed region well under a second"}})
        del step, keep
        torch.cuda.empty_cache()
    # memory-bound kernels at the row lengths of config 5 (layer norm rows of 2048) and config 3 (softmax rows of 512);
    # the layer norm runs on four times config 5's tokens so that its input (268 MB) is larger than L2
    lay = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 8)]), [("batch", "all")])
    B, L, D = 256, 256, 2048
    x, dy = to_device(si.normal(5, "x", [B, L, D], "bf16")), to_device(si.normal(5, "dy", [B, L, D], "bf16"))
    g, b = to_device(si.normal(5, "g", [D], "f32", 0.1, 1.0)), to_device(si.normal(5, "b", [D], "f32", 0.1))
    yb, dxb = torch.empty_like(x), torch.empty_like(x)
    stats = torch.empty(B, L, 2, dtype=torch.float32, device="cuda")
    dg, db = torch.empty_like(g), torch.empty_like(b)
    act = ["batch", "length", "d_model"]
    Nn = mtf.named
    rows = []
    # (the descriptors are built once, outside the timed calls: a call is then a few microseconds of host work,
    #  well under the kernels' durations, so the event pair measures the device)
    nx, ndy, ng, nb, ny, ndx = Nn(x, act), Nn(dy, act), Nn(g, ["d_model"]), Nn(b, ["d_model"]), Nn(yb, act), Nn(dxb, act)
    nst, ndg, ndb = Nn(stats, ["batch", "length", "stat"]), Nn(dg, ["d_model"]), Nn(db, ["d_model"])
    ms = timer(lambda: mtf.mtf_layernorm_forward(lay, nx, ng, nb, 1e-6, ny, nst), 50, stream)
    rows.append(("layernorm_fwd_rows_kernel", f"{B * L} rows of {D}", 2 * x.numel() * 2, ms))
    lnws = torch.empty(max(mtf.mtf_layernorm_workspace_bytes(D), 16), dtype=torch.uint8, device="cuda")
    ms = timer(lambda: mtf.mtf_layernorm_backward(lay, ndy, nx, nst, ng, None, ndx, ndg, ndb, lnws), 50, stream)
    rows.append(("layernorm_bwd_rows_kernel + colsum_finalize_kernel", f"{B * L} rows of {D}, dgamma / dbeta finished in a fixed order", 3 * x.numel() * 2, ms))
    Bs, H, Ls = 16, 16, 512
    names = ["batch", "heads", "length", "memory_length"]
    lg = to_device(si.normal(6, "lg", [Bs, H, Ls, Ls], "f32", 2.0))
    dP = to_device(si.normal(6, "dP", [Bs, H, Ls, Ls], "f32"))
    Pw, dlg = torch.empty(Bs, H, Ls, Ls, dtype=torch.bfloat16, device="cuda"), torch.empty(Bs, H, Ls, Ls, dtype=torch.bfloat16, device="cuda")
    nlg, ndP, nPw, ndlg = Nn(lg, names), Nn(dP, names), Nn(Pw, names), Nn(dlg, names)
    ms = timer(lambda: mtf.mtf_softmax_forward(lay, nlg, False, nPw), 50, stream)
    rows.append(("softmax_fwd_kernel", f"{Bs * H * Ls} rows of {Ls}", lg.numel() * (4 + 2), ms))
    ms = timer(lambda: mtf.mtf_softmax_backward(lay, nPw, ndP, ndlg), 50, stream)
    rows.append(("softmax_bwd_kernel", f"{Bs * H * Ls} rows of {Ls}", lg.numel() * (2 + 4 + 2), ms))
    mtf.mtf_device_status()
    del lg, dP, Pw, dlg
    torch.cuda.empty_cache()
    # ---- the vocab dimension: embedding + logits + cross-entropy, forward and backward, vocab 32768, d_model 1024, tokens 8192
    import numpy as np
    Bv, Lv, Dv, V = 32, 256, 1024, 32768
    Tv = Bv * Lv
    layv = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 8)]), [("vocab", "all")])
    rng = np.random.RandomState(7)
    ids = torch.from_numpy(rng.randint(0, V, size=(Bv, Lv)).astype(np.int32)).cuda()
    tgt = torch.from_numpy(rng.randint(0, V, size=(Bv, Lv)).astype(np.int32)).cuda()
    E, Wo = to_device(si.normal(7, "E", [V, Dv], "bf16")), to_device(si.normal(7, "wout", [Dv, V], "bf16", Dv ** -0.5))
    xv, lgt = torch.empty(Bv, Lv, Dv, dtype=torch.bfloat16, device="cuda"), torch.empty(Bv, Lv, V, dtype=torch.bfloat16, device="cuda")
    lse, loss = torch.empty(Bv, Lv, dtype=torch.float32, device="cuda"), torch.empty(Bv, Lv, dtype=torch.float32, device="cuda")
    dls = torch.full((Bv, Lv), 1.0 / Tv, dtype=torch.float32, device="cuda")
    dhv, dWo, dE = torch.empty_like(xv), torch.empty(Dv, V, dtype=torch.float32, device="cuda"), torch.empty(V, Dv, dtype=torch.float32, device="cuda")
    wsv = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    av, lv, tl = ["batch", "length", "d_model"], ["batch", "length", "vocab"], ["batch", "length"]

    def vocab_step():
        mtf.mtf_embedding_forward(layv, ids, Nn(E, ["vocab", "d_model"]), Nn(xv, av))
        mtf.mtf_xent_forward(layv, Nn(xv, av), Nn(Wo, ["d_model", "vocab"]), tgt, Nn(lgt, lv), Nn(lse, tl), Nn(loss, tl), wsv)
        mtf.mtf_xent_backward(layv, Nn(xv, av), Nn(Wo, ["d_model", "vocab"]), tgt, Nn(lgt, lv), Nn(lse, tl), Nn(dls, tl), Nn(dhv, av), Nn(dWo, ["d_model", "vocab"]), wsv)
        mtf.mtf_embedding_backward(layv, ids, Nn(dhv, av), Nn(dE, ["vocab", "d_model"]))

    ms = timer(vocab_step, 10, stream)
    mtf.mtf_device_status()
    vflops = 6.0 * Tv * Dv * V
    tf = vflops / (ms * 1e-3) / 1e12
    out.append({"metric": "vocab_embedding_logits_xent_fwd_bwd_tflops", "value": tf, "unit": UNIT, "ms_per_step": ms, "dtype": "bf16", "data": "synthetic (seeded)",
                "config": {"workload": f"embedding + logits + softmax cross-entropy, fwd+bwd: tokens={Tv} d_model={Dv} vocab={V}", "mesh": [["all", 8]],
                           "rules": [["vocab", "all"]], "flops_per_step": vflops, "flops_note": "three contractions of 2 tokens d_model vocab"},
                "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_burst"], "frac": tf / peaks["bf16_burst"], "unit": "TFLOP/s",
                             "note": "whole step (3 contractions + 4 memory-bound kernels) against the burst torch.matmul rate"}})
    # the memory-bound kernels of that step, each alone
    nE, nxv, nlgt, nlse, nloss, ndls = Nn(E, ["vocab", "d_model"]), Nn(xv, av), Nn(lgt, lv), Nn(lse, tl), Nn(loss, tl), Nn(dls, tl)
    # (the lookup alone on 16 times the step's tokens, so that it moves more than L2 holds)
    Tg = 16 * Tv
    ids_g = torch.from_numpy(rng.randint(0, V, size=(16 * Bv, Lv)).astype(np.int32)).cuda()
    xg = torch.empty(16 * Bv, Lv, Dv, dtype=torch.bfloat16, device="cuda")
    nxg = Nn(xg, av)
    ms = timer(lambda: mtf.mtf_embedding_forward(layv, ids_g, nE, nxg), 50, stream)
    rows.append(("embedding_gather_kernel", f"{Tg} rows of {Dv} (bf16) from a table of {V} rows (the 67 MB table stays in L2: the reads are L2 hits)", 2 * Tg * Dv * 2, ms))
    del xg, ids_g
    mtf.mtf_xent_forward(layv, Nn(xv, av), Nn(Wo, ["d_model", "vocab"]), tgt, Nn(lgt, lv), Nn(lse, tl), Nn(loss, tl), wsv)
    ms = timer(lambda: mtf.mtf_softmax_xent_forward(layv, nlgt, tgt, nlse, nloss), 20, stream)
    rows.append(("xent_rows_kernel", f"{Tv} rows of {V} (bf16 logits)", Tv * V * 2, ms))
    ms = timer(lambda: mtf.mtf_softmax_xent_backward(layv, nlgt, tgt, nlse, ndls), 20, stream)
    rows.append(("xent_backward_kernel", f"{Tv} rows of {V} (bf16, in place)", Tv * V * 4, ms))
    del lgt, dWo, dE, E, Wo, nE, nlgt
    torch.cuda.empty_cache()
    # Algorithm 1 line 3 on the largest parameter of config 4 (d_model 1024 x d_ff 65536): momentum + weight decay + bf16 working copy
    Dw, Fw = 1024, 65536
    wm = to_device(si.normal(8, "w", [Dw, Fw], "f32", Dw ** -0.5))
    gw = to_device(si.normal(8, "g", [Dw, Fw], "f32", 1e-3))
    mo, wb16 = torch.zeros_like(wm), torch.empty(Dw, Fw, dtype=torch.bfloat16, device="cuda")
    wn2 = ["d_model", "d_ff"]
    layu = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 16)]), [("d_ff", "all")])
    ngw, nwm, nmo, nwb = Nn(gw, wn2), Nn(wm, wn2), Nn(mo, wn2), Nn(wb16, wn2)
    ms = timer(lambda: mtf.mtf_update(layu, ngw, nwm, nmo, nwb, 1e-3, 0.9, 0.01), 20, stream)
    rows.append(("sgd_update_kernel", f"{Dw} x {Fw} f32 parameter with momentum and bf16 copy", Dw * Fw * 22, ms))
    del wm, gw, mo, wb16, ngw, nwm, nmo, nwb
    torch.cuda.empty_cache()
    # Section 6.1: the block transpose between a batch split and a heads split, [batch, length, heads, d_k] -> [batch, heads, length, d_k]
    Bt, Lt, Ht, Kt = 256, 256, 32, 64
    qt = to_device(si.normal(9, "q", [Bt, Lt, Ht, Kt], "bf16"))
    qo = torch.empty(Bt, Ht, Lt, Kt, dtype=torch.bfloat16, device="cuda")
    nqt, nqo = Nn(qt, ["batch", "length", "heads", "d_k"]), Nn(qo, ["batch", "heads", "length", "d_k"])
    ms = timer(lambda: mtf.mtf_transpose(lay, nqt, nqo), 20, stream)
    rows.append(("permute_copy_kernel", f"[{Bt}, {Lt}, {Ht}, {Kt}] bf16 -> [batch, heads, length, d_k]", 2 * qt.numel() * 2, ms))
    xt2 = qt.view(Bt * Lt, Ht * Kt)
    xo2 = qo.view(Ht * Kt, Bt * Lt)
    nxt2, nxo2 = Nn(xt2, ["tokens", "d_model"]), Nn(xo2, ["d_model", "tokens"])
    ms = timer(lambda: mtf.mtf_transpose(lay, nxt2, nxo2), 20, stream)
    rows.append(("permute_transpose_kernel", f"[{Bt * Lt}, {Ht * Kt}] bf16 -> [d_model, tokens]", 2 * qt.numel() * 2, ms))
    mtf.mtf_device_status()
    # the generic kernel (config 1: the fp32 example of Section 8 on mesh [2,2]; parity path, never tuned) and the slice gather
    lay1 = mtf.mtf_layout(mtf.mtf_mesh_create([("rows", 2), ("cols", 2)]), [("batch", "rows"), ("hidden", "cols")])
    x1, w1 = to_device(si.normal(0, "x", [8, 64], "f32")), to_device(si.normal(0, "w", [64, 256], "f32", 0.125))
    h1 = torch.empty(8, 256, dtype=torch.float32, device="cuda")
    nx1, nw1, nh1 = Nn(x1, ["batch", "io"]), Nn(w1, ["io", "hidden"]), Nn(h1, ["batch", "hidden"])
    ms = timer(lambda: mtf.mtf_einsum(lay1, None, [nx1, nw1], nh1, None), 50, stream)
    out.append({"metric": "einsum_simt_kernel_ms", "kernel": "einsum_simt_kernel", "value": ms, "unit": "ms", "ms": ms,
                "config": {"workload": "config 1: x[8, 64] . w[64, 256] in fp32 on mesh [2,2] (131072 multiply-adds: launch-bound)"},
                "roofline": {"bound": "alu", "achieved": 2.0 * 8 * 64 * 256 / (ms * 1e-3) / 1e12, "peak": 148 * 128 * 2 * 1.965e9 / 1e12, "unit": "TFLOP/s",
                             "frac": 2.0 * 8 * 64 * 256 / (ms * 1e-3) / (148 * 128 * 2 * 1.965e9),
                             "note": "fp32 FMA peak = 148 SMs x 128 lanes x 2 flop x 1.965 GHz; a 0.26 MFLOP problem measures launch latency only"}})
    gl = mtf.mtf_layout(mtf.mtf_mesh_create([("all", 8)]), [("d_ff", "all")])
    gsrc = torch.empty(32768, 8192, dtype=torch.bfloat16, device="cuda")
    gdst = torch.empty(32768, 1024, dtype=torch.bfloat16, device="cuda")
    ngs = Nn(gsrc, ["tokens", "d_ff"])
    ms = timer(lambda: mtf.mtf_slice_gather(gl, ngs, 3, gdst), 20, stream)
    rows.append(("mtf_slice_gather (permute_copy_kernel)", "processor 3's slice [32768, 1024] of a bf16 [32768, 8192] tensor (d_ff split 8 ways)", 2 * gdst.numel() * 2, ms))
    mtf.mtf_device_status()
    for kernel, shape, nbytes, ms in rows:
        gbs = nbytes / (ms * 1e-3) / 1e9
        out.append({"metric": "row_kernel_gbs", "kernel": kernel, "value": gbs, "unit": "GB/s", "ms": ms, "config": {"workload": shape},
                    "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"], "unit": "GB/s",
                                 "algorithmic_bytes": nbytes, "note": "read every input once, write every output once; inputs larger than L2"}})
    return out


def run_block(args):
    """Times mtf_attention_* (config 3) or mtf_decoder_layer_* (config 5) forward + backward on one GPU, on seeded
    inputs, and prints one JSON line (this leg measures time only, parity is the tests' job)."""
    import torch
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    import paper_1811_02084_b200 as mtf
    dec = args.workload == "decoder"
    step, flops, desc, keep = block_step(mtf, dec, args.batch if args.batch != 32 else None)
    stream = torch.cuda.current_stream()
    n0 = None
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = mtf.mtf_launch_count()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    mtf.mtf_device_status()
    ms = e0.elapsed_time(e1) / args.steps
    print(json.dumps({"metric": f"transformer_{args.workload}_fwd_bwd_tflops", "value": flops / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16",
                      "data": "synthetic (seeded)", "gpu_launches": mtf.mtf_launch_count() - n0, "config": desc}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layout", default="mp8", choices=sorted(LAYOUTS))
    ap.add_argument("--split", default="dp", choices=["dp", "mp"], help="with N > 1 GPUs: which dimension the rank-spanning mesh dimension takes (dp: batch, mp: d_ff)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the extra two-second back-to-back run")
    ap.add_argument("--no-secondary", action="store_true", help="skip the records of the other workloads and of the memory-bound kernels")
    ap.add_argument("--d-ff", type=int, default=WORKLOAD["d_ff"], help="4096 = config 2, 65536 (with --layout mp16) = config 4")
    ap.add_argument("--batch", type=int, default=WORKLOAD["batch"], help="sequences of 256 tokens per GPU (smaller only for profiler captures)")
    ap.add_argument("--main-only", action="store_true", help="skip the per-layout table and the end-to-end leg (profiler captures)")
    ap.add_argument("--workload", default="ffn", choices=["ffn", "attention", "decoder", "rowkernels"],
                    help="ffn = the headline line; attention / decoder print a secondary line; rowkernels runs the memory-bound kernels only (a few launches each, for profiler captures)")
    args = ap.parse_args()
    WORKLOAD["batch"] = args.batch
    WORKLOAD["d_ff"] = args.d_ff
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "rowkernels":
        import torch
        assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
        import paper_1811_02084_b200 as mtf
        print(json.dumps({"metric": "row_kernels", "records": run_secondary(mtf, measured_peaks(), blocks=False, reps=args.steps if args.steps < 10 else None)}), flush=True)
    elif args.workload != "ffn":
        run_block(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
