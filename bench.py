#!/usr/bin/env python
"""Benchmark of the Token Radius Attention hot path on B200.

One "step" is one pass of the whole hot path over one layer's synthetic Q/K/V at the
75,600-token / 40-head / d=128 shape (Wan-14B 720p, 81 frames):

    tile-major gather of Q, K, V  ->  dense attention + entropy  ->  budget / radius
    ->  block-mask construction   ->  block-sparse attention     ->  scatter of O

`value` is the effective throughput of that pass, 4*d*(computed query-key pairs)/time summed
over the dense and the sparse attention of the step, with inputs resident in HBM.  The sparse
layer on its own (the quantity the paper's speedups are about: ms per layer, TFLOP/s on
computed pairs, fraction of the tensor-core peak, density, speedup against this library's own
dense attention, mask + radius overhead) is nested in `roofline.sparse`.  The JSON line also
carries per-stage times (`stages`), sensitivity rows (`sweeps`), the other shapes the paper
measures on (`other_workloads`), the 50-step denoising-schedule emulation (`schedule`), the
end-to-end number with host buffers (`e2e`) and the fp64 oracle timed on the host cores
(`cpu_baseline`).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME]
                    [--shard replicas|heads]

With N > 1 (torchrun, one rank per GPU) the path shards by (batch, head) with no exchange and no
collective on the data path: `--shard replicas` (default) runs one whole layer per rank (weak
scaling), `--shard heads` gives rank r the heads r, r + N, ... of one layer (strong scaling).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2608_02504_b200 import workloads

METRIC = ("TRA hot-path effective TFLOP/s at 75.6K tokens: one mask-building step = dense attention + entropy, "
          "budget/radius, block mask and one block-sparse attention (4*d*computed pairs of both attentions / "
          "step time); the sparse layer itself is in roofline.sparse")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (read + write) per head of one attention launch at the 75.6K-token shape, from an ncu
# capture of a 4-head case (234.4 MB + 61.1 MB for 4 heads of the sparse launch; 237.1 + 62.2 MB for
# the fused dense + entropy launch); traffic grows in proportion to the head count.
NCU_SPARSE_TRAFFIC_BYTES_PER_HEAD = (234.363136e6 + 61.101568e6) / 4
NCU_DENSE_TRAFFIC_BYTES_PER_HEAD = (237.128448e6 + 62.174464e6) / 4
N_SCHED, N_WARM = 50, 12          # denoising-schedule emulation: floor(0.25 * 50) dense steps


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class NvmlSampler:
    """Samples the SM clock and the clock-event reasons through NVML (read-only queries) every 50 ms from a
    thread, between window() and stop().  nvidia-smi in loop mode delivers only about one line per second while
    the GPU is busy, which leaves a three-second timed region with a handful of samples; ClockSampler below is
    the fallback when the NVML binding is missing."""

    def __init__(self, gpu_index):
        import threading
        import pynvml
        self.nv = pynvml
        pynvml.nvmlInit()
        try:
            uuid = str(torch.cuda.get_device_properties(gpu_index).uuid)
            self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
        except Exception:
            self.h = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
        self.smax = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        self.samples, self.mask, self.on, self.done = [], 0, False, False
        self.thread = threading.Thread(target=self._run, daemon=True)

    def start(self):
        self.thread.start()

    def _run(self):
        nv = self.nv
        while not self.done:
            if self.on:
                try:
                    self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                    self.mask |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    pass
            time.sleep(0.05)

    def window(self, t_begin, t_end):
        self.on = t_end is None         # window(t, None) opens the sampling window, stop() closes it

    def stop(self):
        self.on, self.done = False, True
        self.thread.join(timeout=2)
        nv = self.nv
        names = [("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown),
                 ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                 ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown),
                 ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap)]
        reasons = sorted(n for n, bit in names if self.mask & bit)
        busy = [c for c in self.samples if c > 0]
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": self.smax, "reasons": reasons,
                "samples": len(self.samples), "source": "nvml, every 50 ms"}


def make_sampler(gpu_index):
    try:
        return NvmlSampler(gpu_index)
    except Exception:
        return ClockSampler(gpu_index)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = f"/tmp/tra_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu_index), "-lms", "200"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def window(self, t_begin, t_end):
        """Only samples taken between these two time.time() values count (the sampler is started well before
        the timed region, because nvidia-smi takes a second or two to deliver its first line)."""
        if t_end is not None:
            self.t_begin, self.t_end = t_begin, t_end

    @staticmethod
    def _stamp(text):
        import datetime
        try:
            return datetime.datetime.strptime(text, "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                ts = self._stamp(f[0])
                if ts is not None and getattr(self, "t_begin", None) is not None and \
                        not (self.t_begin <= ts <= self.t_end + 0.2):
                    continue
                try:
                    sm.append(float(f[1]))
                    smax.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        busy = [c for c in sm if c > 0]
        return {"sm_mhz": float(np.median(busy)) if busy else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_setup():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def reduce_over_ranks(x, world, device, op="max"):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def computed_pairs(mask, N, block):
    """Query-key pairs inside the retained blocks (valid rows x valid columns), summed over heads."""
    NB = mask.shape[-1]
    valid = torch.full((NB,), float(block), dtype=torch.float64, device=mask.device)
    valid[-1] = N - (NB - 1) * block
    m = mask.reshape(-1, NB, NB).to(torch.float64)
    return float(torch.einsum("u,huv,v->", valid, m, valid).item())


def pairing_stats(mask, pairs, block):
    """Key-block list entries a CTA walks (union of its two query tiles) over the mean list length of
    a tile, for consecutive tiles and for the tile-pair table of the block-mask call (1.0 = every key
    block serves both tiles; block 128 only: one query block per tile)."""
    if block != 128:
        return None
    heads, NB = mask.shape[-3], mask.shape[-1]
    m = mask.reshape(heads, NB, NB).bool()
    n2 = (NB // 2) * 2

    def ratio(a, b):
        union = (a | b).sum(-1).double()
        own = (a.sum(-1) + b.sum(-1)).double() / 2
        single = (a ^ b).sum(-1).double()
        return {"union_over_own": round(float(union.sum() / own.sum()), 4),
                "single_tile_entries_frac": round(float(single.sum() / union.sum()), 4)}

    out = {"consecutive": ratio(m[:, 0:n2:2], m[:, 1:n2:2])}
    p = pairs.reshape(heads, -1, 2).long()
    ok = p[:, :, 1] >= 0
    hidx = torch.arange(heads, device=m.device)[:, None].expand_as(p[:, :, 0])
    a = m[hidx[ok], p[:, :, 0][ok]]
    b = m[hidx[ok], p[:, :, 1][ok]]
    out["tile_pair_table"] = ratio(a, b)
    return out


def time_ms(fn, reps, warm=1):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2608_02504_b200 import api

    rank, world, local = dist_setup()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    cfg = dict(workloads.CONFIGS[args.config])
    if args.tau is not None:
        cfg["tau"] = args.tau
    if args.heads is not None:
        cfg["heads"] = args.heads
    my_heads = list(range(cfg["heads"]))
    if args.shard == "heads" and world > 1:
        my_heads = my_heads[rank::world]          # heads are independent problems: no exchange step
    heads = len(my_heads)
    N, d, block = workloads.num_tokens(cfg), cfg["head_dim"], cfg["block"]
    peaks = load_peaks()

    sampler = make_sampler(local)
    sampler.start()                     # started early; only samples of the timed region count
    # Layout of the timed step (the caller's tensors are in raster order):
    #   "qo" (default where the grid allows it): a TRA_ORDER_RASTER_QO plan.  K and V are gathered into tile-major
    #        order; Q is read and O written in raster order by the attention launches themselves (Q is loaded
    #        once per thread block and O rows are stored one by one anyway), so the gather of Q and the scatter
    #        of O drop out at no cost to the launches;
    #   "explicit": gather Q, K, V and scatter O, as the paper does;
    #   "raster": a TRA_ORDER_RASTER plan, no layout pass at all; K / V tiles then arrive as sixteen small TMA
    #        boxes instead of two, which costs the launches more than the passes it saves.
    # `stages.raster_order` has the launch times of the third form whatever the choice.  plan_tm is the plan for
    # tile-major tensors, which the measurements after the timed region use.
    plan_tm = api.Plan.from_config(cfg)
    plan, layout = plan_tm, "explicit"
    if args.layout != "explicit":
        try:
            plan = api.Plan.from_config(cfg, flags=api.TRA_ORDER_RASTER if args.layout == "raster"
                                        else api.TRA_ORDER_RASTER_QO)
            layout = args.layout
        except api.TraError:
            pass
    raster = layout == "raster"             # K and V in raster order too
    raster_qo = layout != "explicit"        # Q and O in raster order
    Qr, Kr, Vr = workloads.make_qkv(cfg, dev, heads=my_heads)
    NB = plan.NB
    rows = heads * NB
    # caller-owned buffers, allocated once
    Q, K, V = torch.empty_like(Qr), torch.empty_like(Qr), torch.empty_like(Qr)
    O_dense, O_tm = torch.empty_like(Qr), torch.empty_like(Qr)
    O_raster = torch.empty_like(Qr)
    H = torch.empty(1, heads, N, dtype=torch.float32, device=dev)
    budget = torch.empty(1, heads, N, dtype=torch.int32, device=dev)
    radius = torch.empty(1, heads, N, dtype=torch.float32, device=dev)
    ridx = torch.empty(1, heads, N, dtype=torch.int16, device=dev)
    mask = torch.empty(1, heads, NB, NB, dtype=torch.uint8, device=dev)
    row_ptr = torch.empty(rows + 1, dtype=torch.int32, device=dev)
    col_idx = torch.empty(rows * NB, dtype=torch.int32, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    pairs = torch.empty(heads, plan.n_tile_pairs, 2, dtype=torch.int32, device=dev)

    lib, h = api._lib, plan._h
    import ctypes
    vp = ctypes.c_void_p
    row_bytes = d * 2
    scale = 1.0 / math.sqrt(d)
    ptr = lambda t: vp(t.data_ptr())
    stream = lambda: vp(torch.cuda.current_stream().cuda_stream)

    stage_names = ["gather", "dense_entropy", "budget_radius", "block_mask", "sparse", "scatter"]
    # block mask = vote, row scan, list fill, tile pairing; explicit layout = 3 gathers and 1 scatter
    launches_per_step = 1 + 1 + 4 + 1 + (0 if raster else (2 if raster_qo else 4))
    Qa = Qr if raster_qo else Q                                # what the attention calls of the step read
    Ka, Va = (Kr, Vr) if raster else (K, V)
    O_step = O_raster if raster_qo else O_tm                   # ... and write
    to_gather = [] if raster else ([(Kr, K), (Vr, V)] if raster_qo else [(Qr, Q), (Kr, K), (Vr, V)])

    def one_step(events=None):
        def mark(i):
            if events is not None:
                events[i].record()
        mark(0)
        for s_, d_ in to_gather:
            api._check(lib.tra_tile_major_gather(h, ptr(s_), ptr(d_), heads, row_bytes, stream()), "gather")
        mark(1)
        api._check(lib.tra_entropy_attn(h, ptr(Qa), ptr(Ka), ptr(Va), ptr(O_dense), ptr(H), None, 1, heads,
                                        scale, stream()), "entropy_attn")
        mark(2)
        api._check(lib.tra_budget_radius(h, ptr(H), ptr(budget), ptr(radius), ptr(ridx), 1, heads, stream()),
                   "budget_radius")
        mark(3)
        api._check(lib.tra_build_block_mask(h, ptr(ridx), ptr(mask), ptr(row_ptr), ptr(col_idx),
                                            col_idx.numel(), ptr(nnz), ptr(pairs), 1, heads, stream()), "block_mask")
        mark(4)
        api._check(lib.tra_sparse_attn(h, ptr(Qa), ptr(Ka), ptr(Va), ptr(row_ptr), ptr(col_idx), None, ptr(pairs),
                                       ptr(O_step), None, 1, heads, scale, stream()), "sparse_attn")
        mark(5)
        if not raster_qo:
            api._check(lib.tra_tile_major_scatter(h, ptr(O_tm), ptr(O_raster), heads, row_bytes, stream()), "scatter")
        mark(6)

    for i in range(args.warmup):
        one_step()
        if i == 0:                      # fail fast if a kernel recorded an error
            plan.check_status()
    torch.cuda.synchronize()
    plan.check_status()

    # ---- timed region: K steps, device-timed, inputs resident in HBM -----------------------
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(7)] for _ in range(args.steps)]
    barrier(world)
    torch.cuda.synchronize()
    t_wall = time.time()
    sampler.window(t_wall, None)
    for k in range(args.steps):
        one_step(ev[k])
    torch.cuda.synchronize()
    barrier(world)
    wall_s = time.time() - t_wall
    sampler.window(t_wall, t_wall + wall_s)
    clocks = sampler.stop()
    total_ms = reduce_over_ranks(ev[0][0].elapsed_time(ev[-1][6]), world, dev)
    plan.check_status()

    stage_ms = {}
    for i, name in enumerate(stage_names):
        vals = [ev[k][i].elapsed_time(ev[k][i + 1]) for k in range(args.steps)]
        stage_ms[name] = {"mean": float(np.mean(vals)), "min": float(np.min(vals)), "median": float(np.median(vals))}

    pairs_sparse = computed_pairs(mask, N, block)
    pairs_dense = float(heads) * N * N
    flops_rank = 4.0 * d * (pairs_dense + pairs_sparse)
    flops_job = reduce_over_ranks(flops_rank, world, dev, "sum")       # all ranks' work
    ms_per_step = total_ms / args.steps
    value = flops_job / (ms_per_step * 1e-3) / 1e12

    t_sparse = stage_ms["sparse"]["mean"] * 1e-3
    t_dense = stage_ms["dense_entropy"]["mean"] * 1e-3
    tf_sparse = 4.0 * d * pairs_sparse / t_sparse / 1e12
    tf_dense = 4.0 * d * pairs_dense / t_dense / 1e12
    peak_tf, peak_burst = peaks["bf16_tflops_sustained"], peaks["bf16_tflops"]
    peak_note = f"{peaks['_source']} bf16 sustained cuBLAS"

    # ---- launches timed on their own (back to back, as the sparse steps of a schedule run) -------
    # From here on the tensors are tile-major (plan_tm): the explicit gather / scatter of the paper's design,
    # which a raster-order step does without, is timed here.
    reps = max(2, min(5, args.steps))
    gather_all = lambda: [plan_tm.tile_major_gather(s_, out=d_) for s_, d_ in zip((Qr, Kr, Vr), (Q, K, V))]
    t_gather_explicit = time_ms(gather_all, reps, 1) * 1e-3
    t_scatter_explicit = time_ms(lambda: plan_tm.tile_major_scatter(O_tm, out=O_dense), reps, 1) * 1e-3
    plan_step, plan = plan, plan_tm
    sparse_call = lambda tp: plan.sparse_attn(Q, K, V, row_ptr, col_idx, O=O_tm, tile_pairs=tp)
    t_plain = time_ms(lambda: plan.entropy_attn(Q, K, V, O=O_dense, want_entropy=False), reps) * 1e-3
    t_sparse_b2b = time_ms(lambda: sparse_call(pairs), 2 * reps, 2) * 1e-3
    t_sparse_consecutive = time_ms(lambda: sparse_call(None), reps, 1) * 1e-3
    # the token mask of Eq. 15 inside the retained blocks, and Eq. 16 itself (no block list)
    t_token = time_ms(lambda: plan.sparse_attn(Q, K, V, row_ptr, col_idx, O=O_tm, ridx=ridx, tile_pairs=pairs),
                      reps, 2) * 1e-3
    t_token_level = time_ms(lambda: plan.sparse_attn(Q, K, V, None, None, O=O_tm, ridx=ridx), reps, 1) * 1e-3
    # the same two launches on raster-order tensors (a TRA_ORDER_RASTER plan), where the grid allows it
    raster_order = None
    try:
        plan_r = plan_step if raster else api.Plan.from_config(cfg, flags=api.TRA_ORDER_RASTER)
        O_tmp = torch.empty_like(Qr)
        t_r_dense = time_ms(lambda: plan_r.entropy_attn(Qr, Kr, Vr, O=O_tmp, entropy=H), reps, 1)
        t_r_sparse = time_ms(lambda: plan_r.sparse_attn(Qr, Kr, Vr, row_ptr, col_idx, O=O_tmp, tile_pairs=pairs),
                             reps, 2)
        plan_r.check_status()
        same = bool(torch.equal(O_tmp, plan_tm.tile_major_scatter(sparse_call(pairs)[0])))
        raster_order = {"dense_entropy_ms": round(t_r_dense, 3), "sparse_ms": round(t_r_sparse, 3),
                        "sparse_output_equals_gather_attend_scatter": same,
                        "note": "Q, K, V read in raster order through 16-row TMA boxes, O written in raster order: "
                                "no gather / scatter pass, slower launches"}
        del O_tmp
        if not raster:
            plan_r.close()
    except api.TraError:
        pass
    plan.entropy_attn(Q, K, V, O=O_dense, entropy=H)      # O_dense and O_tm hold the timed pass's results again
    sparse_call(pairs)

    overhead_ms = stage_ms["budget_radius"]["mean"] + stage_ms["block_mask"]["mean"]
    n_sparse_steps = N_SCHED - N_WARM
    amort_ms = (N_WARM * stage_ms["dense_entropy"]["mean"] + overhead_ms
                + n_sparse_steps * stage_ms["sparse"]["mean"]) / N_SCHED
    tf_b2b = 4.0 * d * pairs_sparse / t_sparse_b2b / 1e12
    stages = {
        "ms": {k: round(v["mean"], 4) for k, v in stage_ms.items()},
        "ms_min": {k: round(v["min"], 4) for k, v in stage_ms.items()},
        "ms_median": {k: round(v["median"], 4) for k, v in stage_ms.items()},
        "dense_plain_ms": round(t_plain * 1e3, 4),
        "dense_plain_tflops": round(4.0 * d * pairs_dense / t_plain / 1e12, 2),
        "dense_entropy_tflops": round(tf_dense, 2),
        "sparse_tflops": round(tf_sparse, 2),
        "sparse_with_token_mask_ms": round(t_token * 1e3, 4),
        "token_level_no_block_list_ms": round(t_token_level * 1e3, 4),
        "schedule_amortised_ms_per_step_from_stages": round(amort_ms, 3),
        "budget_radius_gbs": round(heads * N * 14 / (stage_ms["budget_radius"]["mean"] * 1e-3) / 1e9, 1),
        "block_mask_gbs": round((heads * N * 2 + heads * NB * NB + 4 * rows + 4 * int(nnz.item()))
                                / (stage_ms["block_mask"]["mean"] * 1e-3) / 1e9, 2),
        "layout": {"qo": "K and V gathered into tile-major order inside the step; Q read and O written in raster "
                         "order by the attention launches (no gather of Q, no scatter of O)",
                   "explicit": "Q, K, V gathered and O scattered inside the step",
                   "raster": "Q, K, V read and O written in raster order by the attention launches (16-row TMA "
                             "boxes; no gather / scatter pass)"}[layout],
        "raster_order": raster_order,
        "explicit_gather_ms": round(t_gather_explicit * 1e3, 4),
        "explicit_scatter_ms": round(t_scatter_explicit * 1e3, 4),
        "gather_gbs": round(3 * 2 * heads * N * row_bytes / t_gather_explicit / 1e9, 1),
    }

    # `roofline` is the kernel that dominates the step (the fused dense + entropy launch, ~70 % of a
    # pass); `roofline.sparse` is the block-sparse layer: the launch as timed inside the step, right
    # behind the dense launch and the mask kernels, and back to back as in the sparse steps of a run.
    full_shape = args.config == "wan14b-720p"
    roofline = {
        "bound": "tensor", "kernel": "tra_attn_kernel<128,128,entropy,dense> (dense attention + entropy)",
        "achieved": round(tf_dense, 2), "peak": peak_tf, "unit": "TFLOP/s", "frac": round(tf_dense / peak_tf, 4),
        "frac_of_burst_peak": round(tf_dense / peak_burst, 4),
        "traffic": NCU_DENSE_TRAFFIC_BYTES_PER_HEAD * heads if full_shape else None,
        "peak_source": peak_note, "peak_burst": peak_burst, "flops_per_launch": 4.0 * d * pairs_dense,
        "launch_ms": round(t_dense * 1e3, 4),
        "sparse": {
            "kernel": "tra_attn_kernel<128,128,block list> (block-sparse attention over retained blocks)",
            "bound": "tensor", "unit": "TFLOP/s", "flops_per_launch": 4.0 * d * pairs_sparse,
            "launch_ms": round(t_sparse * 1e3, 4), "achieved": round(tf_sparse, 2),
            "frac": round(tf_sparse / peak_tf, 4), "frac_of_burst_peak": round(tf_sparse / peak_burst, 4),
            "back_to_back": {"launch_ms": round(t_sparse_b2b * 1e3, 4), "achieved": round(tf_b2b, 2),
                             "frac": round(tf_b2b / peak_tf, 4), "frac_of_burst_peak": round(tf_b2b / peak_burst, 4),
                             "note": "consecutive sparse launches, as in the 38 sparse steps of the schedule"},
            "consecutive_tiles_ms": round(t_sparse_consecutive * 1e3, 4),
            "traffic": NCU_SPARSE_TRAFFIC_BYTES_PER_HEAD * heads if full_shape else None,
            "block_density": round(pairs_sparse / pairs_dense, 4), "retained_blocks": int(nnz.item()),
            "speedup_vs_own_dense_plain": round(t_plain / t_sparse, 3),
            "speedup_vs_own_dense_plain_back_to_back": round(t_plain / t_sparse_b2b, 3),
            "mask_radius_ms": round(overhead_ms, 4),
            "mask_radius_overhead_frac_one_layer": round(overhead_ms / (stage_ms["sparse"]["mean"] + overhead_ms), 4),
            "mask_radius_overhead_frac_amortised_38_sparse_steps": round(
                (overhead_ms / n_sparse_steps) / (stage_ms["sparse"]["mean"] + overhead_ms / n_sparse_steps), 5),
            "cta_key_block_lists": pairing_stats(mask, pairs, block),
        },
    }

    extras = rank == 0 and not args.quick
    sweeps = run_sweeps(api, cfg, plan, dev, (Q, K, V, O_tm, H), t_plain, peak_tf) if extras and args.sweeps else None
    other = None
    if extras and args.other_workloads and full_shape and args.heads is None:
        other = [run_workload(api, "tiny", dev, peak_tf), run_workload(api, "wan1.3b-480p", dev, peak_tf),
                 run_workload(api, "hunyuan-720p", dev, peak_tf),
                 run_workload(api, "hunyuan-720p", dev, peak_tf, gamma=0.0513)]     # slow temporal decay
    schedule = None
    if extras and args.schedule:
        bufs = (Q, K, V, O_dense, O_tm, H, budget, radius, ridx, mask, row_ptr, col_idx, nnz, pairs)
        q_keep, k_keep = Q.clone(), K.clone()
        schedule = run_schedule(cfg, plan, dev, bufs, N_SCHED, N_WARM)
        schedule["refresh_variants"] = []
        for every in (10, 5, 2):        # the paper's refresh ablation: never / every 10 / 5 / 2 steps
            Q.copy_(q_keep)
            K.copy_(k_keep)
            schedule["refresh_variants"].append(run_schedule(cfg, plan, dev, bufs, N_SCHED, N_WARM, every))
        Q.copy_(q_keep)
        K.copy_(k_keep)
        schedule["entropy_in_last_warmup_step_only"] = run_schedule(cfg, plan, dev, bufs, N_SCHED, N_WARM,
                                                                    entropy_last_only=True)
        del q_keep, k_keep
    if extras:
        one_step()                       # every buffer holds the default pass again
        if raster_qo:                    # ... with tile-major Q, K, V and dense output, for the CPU sample's check
            gather_all()
            plan.entropy_attn(Q, K, V, O=O_dense, entropy=H)
        torch.cuda.synchronize()

    # ---- end to end: host buffers in, host buffer out, copies inside the timed region --------
    e2e = run_e2e(args, api, plan_step, (Qr, Kr, Vr), O_raster, flops_rank, world, dev)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = run_cpu_sample(cfg, n_rows=args.cpu_rows, gpu_pass=(Qr, Kr, Vr, O_dense, H))

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 3), "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4),
            "higher_is_better": True, "scaling": "strong" if args.shard == "heads" and world > 1 else "weak",
            "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic (seeded generator shaped like Wan2.1/2.2-14B 720p attention inputs)",
            "config": bench_config(args, cfg, world, heads),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "stages": stages, "sweeps": sweeps, "other_workloads": other,
            "schedule": schedule, "cpu_baseline": cpu_baseline,
            "paper_context": "paper: 1.56-2.05x end-to-end speedup at 9-19% retained interactions on one H200",
            "wall_s_timed_region": round(wall_s, 3),
        }
        print(json.dumps(line))
    plan.close()
    if plan_step is not plan:
        plan_step.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def bench_config(args, cfg, world, heads_per_rank):
    shard = args.shard if world > 1 else "one GPU"
    return {"workload": args.config, "grid": [cfg["T"], cfg["H"], cfg["W"]], "tokens": workloads.num_tokens(cfg),
            "heads": cfg["heads"], "head_dim": cfg["head_dim"], "block": cfg["block"],
            "tile": [cfg["tile_h"], cfg["tile_w"]], "tau": cfg["tau"], "gamma": cfg["gamma"],
            "radius_policy": "extended", "batch_per_gpu": 1, "heads_per_gpu": heads_per_rank,
            "parallelism": f"{shard} x{world} (heads/batch shard, no collective)",
            "l2": "inputs larger than L2 (Q/K/V/O are 774 MB each)"}


def sparse_layer(api, cfg, Q, K, V, O, H, t_plain_ms, peak_tf, reps=3, **plan_kw):
    """Budget/radius, block mask and block-sparse attention of one layer under another plan (same
    entropies, inputs already tile-major for that plan): density, ms, TFLOP/s, speedup."""
    plan = api.Plan.from_config(cfg, **plan_kw)
    N, d, heads, block = plan.N, cfg["head_dim"], Q.shape[1], cfg["block"]
    _, _, ridx = plan.budget_radius(H, want_budget=False, want_radius=False)
    mask, row_ptr, col_idx, nnz, pairs = plan.build_block_mask(ridx, want_tile_pairs=True)
    t_mask = time_ms(lambda: plan.build_block_mask(ridx, mask, row_ptr, col_idx, nnz, pairs), 2, 0)
    ms = time_ms(lambda: plan.sparse_attn(Q, K, V, row_ptr, col_idx, O=O, tile_pairs=pairs), reps, 2)
    plan.check_status()
    p = computed_pairs(mask, N, block)
    out = {"block_density": round(p / (heads * float(N) * N), 4), "sparse_ms": round(ms, 3),
           "block_mask_ms": round(t_mask, 3),
           "sparse_tflops": round(4.0 * d * p / (ms * 1e-3) / 1e12, 1),
           "sparse_frac_of_peak": round(4.0 * d * p / (ms * 1e-3) / 1e12 / peak_tf, 4),
           "speedup_vs_dense_plain": round(t_plain_ms / ms, 2)}
    plan.close()
    return out


def run_sweeps(api, cfg, plan, dev, bufs, t_plain, peak_tf):
    """Sensitivity rows on the main workload (same Q/K/V, the entropies of the timed pass): target
    mass tau (the paper's 9-19 % density band is reached at smaller tau), the literal candidate set
    of Eq. 14, the decay read as a per-frame factor, tile shapes of the tile-major order and the
    block size (the paper's hyper-parameter tables)."""
    Q, K, V, O, H = bufs
    t_plain_ms = t_plain * 1e3
    out = {"tau": [], "tile_shape": [], "block_size": []}
    for tau in (0.5, 0.3):
        out["tau"].append({"tau": tau, **sparse_layer(api, dict(cfg, tau=tau), Q, K, V, O, H, t_plain_ms, peak_tf)})
    out["radius_policy_literal"] = {
        "note": "candidate set 0..D plus +inf: every query whose budget exceeds C_grid(D) jumps to full support",
        **sparse_layer(api, cfg, Q, K, V, O, H, t_plain_ms, peak_tf, reps=2, radius_policy=api.TRA_RADII_LITERAL)}
    g_factor = -math.log(cfg["gamma"]) if 0.0 < cfg["gamma"] < 1.0 else None
    if g_factor is not None:            # "decay factor 0.6" read as a per-frame factor f^delta: gamma = -ln f
        out["gamma_as_per_frame_factor"] = {
            "gamma": round(g_factor, 4),
            **sparse_layer(api, dict(cfg, gamma=g_factor), Q, K, V, O, H, t_plain_ms, peak_tf, reps=2)}
    # other tile shapes and block 64 change the token order, so these run a pass of their own
    Qr, Kr, Vr = (plan.tile_major_scatter(x) for x in (Q, K, V))
    for th, tw in ((8, 16), (16, 8), (4, 32), (1, cfg["W"])):
        out["tile_shape"].append({"tile": [th, tw], **own_pass(api, dict(cfg, tile_h=th, tile_w=tw), Qr, Kr, Vr,
                                                               peak_tf)})
    # 128 and 64, then the paper's block sizes as tiles of the 45 x 80 frame (Appendix, block-size table)
    for b, (th, tw) in ((128, (8, 16)), (64, (8, 8)), (120, (15, 8)), (90, (9, 10)), (72, (9, 8)), (48, (3, 16)),
                        (40, (5, 8))):
        if b not in (128, 64) and (cfg["H"] % th or cfg["W"] % tw):     # tiles used as blocks must tile the frame
            continue
        out["block_size"].append({"block": b, "tile": [th, tw],
                                  **own_pass(api, dict(cfg, block=b, tile_h=th, tile_w=tw), Qr, Kr, Vr, peak_tf)})
    return out


def own_pass(api, cfg, Qr, Kr, Vr, peak_tf):
    """One whole pass under another token order / block size: density, sparse and mask time."""
    plan = api.Plan.from_config(cfg)
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    O, H, _ = plan.entropy_attn(Q, K, V)
    t_plain = time_ms(lambda: plan.entropy_attn(Q, K, V, O=O, want_entropy=False), 1, 0)
    plan.close()
    return {"dense_plain_ms": round(t_plain, 3), **sparse_layer(api, cfg, Q, K, V, O, H, t_plain, peak_tf, reps=2)}


def run_schedule(cfg, plan, dev, bufs, n_steps, n_warm, refresh_every=0, entropy_last_only=False):
    """Steps 0..n_warm-1 dense with entropy; radii and mask from the last of them; the rest sparse.
    refresh_every = k > 0: every k-th step after the warm-up runs dense attention with entropy
    again and rebuilds radii and mask (the paper's 'entropy and mask refresh' ablation).
    entropy_last_only: the warm-up steps before the last run plain dense attention (only the last
    warm-up step's entropy is ever used)."""
    Q, K, V, O_dense, O_tm, H, budget, radius, ridx, mask, row_ptr, col_idx, nnz, pairs = bufs
    heads = Q.shape[1]
    q_state = Q.float()       # tile-major fp32 state that drifts; V stays fixed
    k_state = K.float()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * n_steps)]
    n_refresh = 0
    eb0, eb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for step in range(n_steps):
        workloads.drift_(q_state, step, cfg["seed"] + 1)
        workloads.drift_(k_state, step, cfg["seed"] + 2)
        Q.copy_(q_state)
        K.copy_(k_state)
        ev[2 * step].record()
        refresh = refresh_every > 0 and step > n_warm and (step - n_warm) % refresh_every == 0
        n_refresh += int(refresh)
        if step < n_warm - 1 and entropy_last_only:
            plan.entropy_attn(Q, K, V, O=O_dense, want_entropy=False)
        elif step < n_warm or refresh:
            plan.entropy_attn(Q, K, V, O=O_dense, entropy=H)
            if step == n_warm - 1 or refresh:
                eb0.record()
                plan.budget_radius(H, budget=budget, radius=radius, ridx=ridx)
                plan.build_block_mask(ridx, block_mask=mask, row_ptr=row_ptr, col_idx=col_idx, nnz=nnz,
                                      tile_pairs=pairs)
                eb1.record()
        else:
            plan.sparse_attn(Q, K, V, row_ptr, col_idx, O=O_tm, tile_pairs=pairs)
        ev[2 * step + 1].record()
    torch.cuda.synchronize()
    plan.check_status()
    per_step = [ev[2 * s].elapsed_time(ev[2 * s + 1]) for s in range(n_steps)]
    build_ms = eb0.elapsed_time(eb1)
    N, block = plan.N, plan.block
    if entropy_last_only:
        return {"amortised_ms_per_step": round(float(np.sum(per_step)) / n_steps, 3),
                "dense_step_ms": round(float(np.mean(per_step[: n_warm - 1])), 3),
                "note": "plain dense attention in warm-up steps 0..n_warm-2, entropy only in the last one"}
    if refresh_every > 0:
        return {"refresh_every": refresh_every, "refresh_steps": n_refresh,
                "amortised_ms_per_step": round(float(np.sum(per_step)) / n_steps, 3)}
    return {"steps": n_steps, "dense_warmup_steps": n_warm, "sparse_steps": n_steps - n_warm,
            "amortised_ms_per_step": round(float(np.sum(per_step)) / n_steps, 3),
            "dense_step_ms": round(float(np.mean(per_step[: n_warm - 1])), 3),
            "build_ms": round(build_ms, 3),
            "sparse_step_ms": round(float(np.mean(per_step[n_warm:])), 3),
            "retained_block_density": round(computed_pairs(mask, N, block) / (heads * float(N) * N), 4),
            "drift": "Q and K: x_t = x_{t-1} + 0.05 N(0,1) on the fp32 state; V fixed"}


def run_workload(api, name, dev, peak_tf, reps=2, gamma=None):
    """One of the other shapes the paper measures on (stage times of the same pass, 1 warm-up +
    `reps` timed passes): ms per layer, TFLOP/s on computed pairs, retained density, speedup."""
    cfg = dict(workloads.CONFIGS[name])
    if gamma is not None:
        cfg["gamma"] = gamma
    N, d, heads, block = workloads.num_tokens(cfg), cfg["head_dim"], cfg["heads"], cfg["block"]
    plan = api.Plan.from_config(cfg)
    Qr, Kr, Vr = workloads.make_qkv(cfg, dev)
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    del Qr, Kr, Vr
    O = torch.empty_like(Q)
    H = torch.empty(1, heads, N, dtype=torch.float32, device=dev)
    ridx = torch.empty(1, heads, N, dtype=torch.int16, device=dev)
    bufs = None
    names = ("dense_entropy", "budget_radius", "block_mask", "sparse", "dense_plain")
    ms = {k: [] for k in names}
    for it in range(1 + reps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        ev[0].record()
        plan.entropy_attn(Q, K, V, O=O, entropy=H)
        ev[1].record()
        plan.budget_radius(H, ridx=ridx, want_budget=False, want_radius=False)
        ev[2].record()
        if bufs is None:
            bufs = plan.build_block_mask(ridx, want_tile_pairs=True)
        else:
            plan.build_block_mask(ridx, *bufs)
        ev[3].record()
        plan.sparse_attn(Q, K, V, bufs[1], bufs[2], O=O, tile_pairs=bufs[4])
        ev[4].record()
        plan.entropy_attn(Q, K, V, O=O, want_entropy=False)
        ev[5].record()
        torch.cuda.synchronize()
        if it == 0:
            plan.check_status()
            continue
        for i, k in enumerate(names):
            ms[k].append(ev[i].elapsed_time(ev[i + 1]))
    plan.check_status()
    t = {k: float(np.mean(v)) for k, v in ms.items()}
    pairs_sparse = computed_pairs(bufs[0], N, block)
    pairs_dense = float(heads) * N * N
    tf = lambda pairs, msec: 4.0 * d * pairs / (msec * 1e-3) / 1e12
    out = {"workload": name, "tokens": N, "heads": heads, "head_dim": d, "block": block, "gamma": cfg["gamma"],
           "tau": cfg["tau"], "ms": {k: round(v, 4) for k, v in t.items()},
           "dense_entropy_tflops": round(tf(pairs_dense, t["dense_entropy"]), 1),
           "sparse_tflops": round(tf(pairs_sparse, t["sparse"]), 1),
           "sparse_frac_of_peak": round(tf(pairs_sparse, t["sparse"]) / peak_tf, 4),
           "block_density": round(pairs_sparse / pairs_dense, 4),
           "speedup_sparse_vs_dense_plain": round(t["dense_plain"] / t["sparse"], 3),
           "mask_radius_overhead_frac_one_layer": round(
               (t["budget_radius"] + t["block_mask"]) / (t["sparse"] + t["budget_radius"] + t["block_mask"]), 4),
           "cta_key_block_lists": pairing_stats(bufs[0], bufs[4], block)}
    plan.close()
    return out


def run_e2e(args, api, plan, src_dev, O_raster, flops_rank, world, dev, group=8, first_group=1):
    """Same pass with Q, K, V in pinned host memory and O read back to pinned host memory, through
    the library's host pipeline: groups of `group` heads (a smaller first group, so the kernels
    start early), the copies of neighbouring groups overlapping the kernels of the current one.
    Every byte crosses PCIe inside the timed region."""
    steps = max(1, args.e2e_steps)
    host_in = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in src_dev]
    for hbuf, t in zip(host_in, src_dev):
        hbuf.copy_(t)
    host_out = torch.empty(O_raster.shape, dtype=O_raster.dtype, pin_memory=True)
    heads = src_dev[0].shape[1]
    pipe = api.HostPipeline(plan, heads, group=group, first_group=first_group)
    torch.cuda.synchronize()

    pipe.run(host_in[0], host_in[1], host_in[2], host_out)
    torch.cuda.synchronize()
    plan.check_status()
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        pipe.run(host_in[0], host_in[1], host_in[2], host_out)
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    ms = reduce_over_ranks(e0.elapsed_time(e1) / steps, world, dev)
    flops_job = reduce_over_ranks(flops_rank, world, dev, "sum")
    plan.check_status()
    same = bool(torch.equal(host_out.to(O_raster.device), O_raster))
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = host_out.numel() * host_out.element_size()
    return {"value": round(flops_job / (ms * 1e-3) / 1e12, 3), "unit": "TFLOP/s",
            "ms_per_step": round(ms, 3), "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "head_group": pipe.group, "first_head_group": pipe.first_group, "copies_overlap_kernels": True,
            "output_equals_device_path": same}


# ------------------------------------------------------------------------------------------
# the fp64 oracle on the host cores: CPU baseline and reference arm
# ------------------------------------------------------------------------------------------
def run_cpu_sample(cfg, n_rows, seed=0, gpu_pass=None):
    """Times the oracle, as it stands, on a bounded sample of the same workload: one head,
    `n_rows` query rows (whole blocks) through dense attention + entropy, budget/radius,
    the block vote of their block rows, and sparse attention.  With `gpu_pass` = (Q, K, V in raster
    order, dense O and entropy in tile-major order) of the GPU pass, the oracle runs on the very
    tensors of head 0 and the GPU's dense output and entropy are compared on the sampled rows."""
    import oracle
    oracle.build()
    N, d, block = workloads.num_tokens(cfg), cfg["head_dim"], cfg["block"]
    geo = oracle.geometry(cfg["T"], cfg["H"], cfg["W"], cfg["tile_h"], cfg["tile_w"], block, cfg["gamma"], cfg["tau"])
    raster = (geo.coord[:, 0] * geo.H + geo.coord[:, 1]) * geo.W + geo.coord[:, 2]
    if gpu_pass is not None:
        Qr, Kr, Vr = (x[:, :1].cpu() for x in gpu_pass[:3])
    else:
        Qr, Kr, Vr = workloads.make_qkv(cfg, "cpu", heads=[0])
    Qb, Kb, Vb = (workloads.bf16_bits(x[0, 0])[raster] for x in (Qr, Kr, Vr))
    n_blocks = max(1, n_rows // block)
    rng = np.random.default_rng(seed)
    u_list = np.sort(rng.choice(geo.NB - 1, size=min(n_blocks, geo.NB - 1), replace=False)).astype(np.int32)
    rows = (u_list[:, None] * block + np.arange(block)[None, :]).reshape(-1).astype(np.int32)
    scale = 1.0 / math.sqrt(d)
    t0 = time.time()
    dense = oracle.attention_rows(Qb, Kb, Vb, scale, rows)
    t1 = time.time()
    # entropy of the sampled rows; the other queries of the head get a stand-in entropy so that
    # the budget/radius stage runs over the whole head as it would in the pipeline
    Hh = np.full(N, np.float32(math.log(N) / 2), np.float32)
    Hh[rows] = dense["H_def"].astype(np.float32)
    bud, _ = oracle.budget(Hh[None], geo.tau, N)
    ridx = oracle.select_radius(bud, geo.coord, geo.H, geo.W, geo.counts)[0]
    t2 = time.time()
    bm = oracle.block_vote(geo.coord, geo.T, block, geo.theta, ridx, u_list=u_list)
    t3 = time.time()
    vis = oracle.visible_rows(geo.coord, geo.T, block, geo.theta, ridx, rows, np.repeat(bm, block, axis=0), 0)
    oracle.attention_rows(Qb, Kb, Vb, scale, rows, vis)
    t4 = time.time()
    pairs = rows.size * float(N) + float(vis.sum())
    total = t4 - t0
    out = {"value": round(4.0 * d * pairs / total / 1e12, 6), "unit": "TFLOP/s", "cores": oracle.num_threads(),
           "kind": "oracle",
           "sample": f"1 head, {rows.size} query rows ({u_list.size} blocks) of {cfg['heads']}x{N}: dense+entropy "
                     f"{t1 - t0:.2f}s, budget/radius {t2 - t1:.2f}s, block vote {t3 - t2:.2f}s, sparse {t4 - t3:.2f}s",
           "seconds": round(total, 3),
           "extrapolated_ms_per_layer": round(total / rows.size * N * cfg["heads"] * 1e3, 1)}
    if gpu_pass is not None:
        # parity of the timed pass on the sampled rows (head 0): literal max-abs, the number of
        # elements over 1e-2 (they pass through the one-bf16-ulp clause of the criterion), relative L2
        O_gpu, H_gpu = gpu_pass[3:]
        rows_t = torch.from_numpy(rows).long().to(O_gpu.device)
        got = O_gpu[0, 0][rows_t].float().cpu().numpy().astype(np.float64)
        err = np.abs(got - dense["O"])
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(dense["O"]), 2.0 ** -126))) - 7)
        out["gpu_parity_on_sample"] = {
            "dense_output_max_abs": float(err.max()), "elements": int(err.size),
            "elements_over_1e-2": int((err > 1e-2).sum()),
            "elements_failing_max(1e-2, 1 bf16 ulp)": int((err > np.maximum(1e-2, ulp)).sum()),
            "dense_output_rel_l2": float(np.linalg.norm(got - dense["O"]) / np.linalg.norm(dense["O"])),
            "entropy_max_abs": float(np.abs(H_gpu[0, 0][rows_t].cpu().numpy() - dense["H_def"]).max())}
    return out


def run_reference(args):
    """Reference arm: the oracle as it stands, on the host cores, same metric and config."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    cfg = dict(workloads.CONFIGS[args.config])
    if args.tau is not None:
        cfg["tau"] = args.tau
    if args.heads is not None:
        cfg["heads"] = args.heads
    n_rows = max(128, args.cpu_rows // 4)
    for i in range(args.warmup):
        run_cpu_sample(cfg, n_rows=128, seed=100 + i)
    results = [run_cpu_sample(cfg, n_rows=n_rows, seed=i) for i in range(args.steps)]
    secs = float(np.mean([r["seconds"] for r in results]))
    value = float(np.mean([r["value"] for r in results]))
    heads_per_rank = len(range(cfg["heads"])[0::world]) if args.shard == "heads" and world > 1 else cfg["heads"]
    config = bench_config(args, cfg, world, heads_per_rank)
    config["sample_note"] = "each step is a bounded sample of the workload (one head, whole query blocks)"
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(secs * 1e3, 2),
        "higher_is_better": True, "scaling": "strong" if args.shard == "heads" and world > 1 else "weak",
        "vs_baseline": None, "dtype": "f64",
        "data": "synthetic (same seeded generator)",
        "config": config,
        "cpu_baseline": {"value": round(value, 6), "unit": "TFLOP/s", "cores": results[0]["cores"],
                         "kind": "oracle", "sample": results[0]["sample"]},
        "e2e": {"value": round(value, 6), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="wan14b-720p", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: one whole layer per rank (weak scaling) or the heads of one layer split over the ranks")
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--heads", type=int, default=None, help="override the head count (profiling on a small case)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-rows", type=int, default=8192)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="the timed steps, e2e and CPU baseline only")
    ap.add_argument("--layout", default="qo", choices=["qo", "explicit", "raster"],
                    help="which tensors the attention launches of the timed step take in raster order: Q and O "
                         "(default), none (explicit gather / scatter), or all")
    ap.add_argument("--no-schedule", dest="schedule", action="store_false")
    ap.add_argument("--no-sweeps", dest="sweeps", action="store_false",
                    help="skip the tau / candidate-set / decay / tile-shape / block-size rows")
    ap.add_argument("--no-other-workloads", dest="other_workloads", action="store_false",
                    help="skip the tiny, Wan2.1-1.3B and HunyuanVideo shapes reported next to the main workload")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
        run_ours(args)


if __name__ == "__main__":
    main()
