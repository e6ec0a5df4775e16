#!/usr/bin/env python
"""Benchmark of the sparse denoising step on B200.

A timed "step" is one refresh cycle of the workload's schedule (refresh interval R, default 2): one full step
(dense joint attention + action-to-future scoring + selection and maps) followed by R-1 sparse steps (pack,
packed joint attention, scatter) that reuse the selection.  `value` is the number of tokens that went through the
joint attention per second, B * (L + (R-1) L') per cycle, summed over ranks.

Two regimes are timed, each over exactly --steps cycles replayed from one CUDA graph, each with its own record of the
sampled SM clocks: `value` is the steady state (the timed cycles follow at least a second of back-to-back replays, so
the 1000 W power cap has settled the clocks), `value_burst` the same cycles after an idle gap (clocks at maximum).
Stage times are taken in long back-to-back loops as well, i.e. in the steady regime.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl swam|reference]

For N > 1 launch through torch.distributed.run (one rank per GPU); a plain `--gpus N` invocation re-launches
itself that way.  Every rank runs its own batch of samples (weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2609_38984_b200 import dist as sd  # noqa: E402
from paper_2609_38984_b200 import workloads as W  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel's launches in one cycle (dense launch + packed
# launch), from the ncu captures summarised in profiles/attn_bf16_tc_*.txt
DOMINANT_KERNEL_DRAM_BYTES = {
    "larger_imagination": int((228.235008 + 57.636608 + 87.190784 + 10.338048) * 1e6),
    "multi_view": int((639.513856 + 198.916352 + 257.552896 + 69.681920) * 1e6),   # profiles/attn_bf16_tc_multi_view.txt
}
N_SMS = 148
EX2_PER_CLK_PER_SM = 16      # ex2.approx.f32: one warp instruction per 8 clk on each of the four sub-cores
STEADY_PRELOAD_S = 1.0       # back-to-back replays before the steady-state timed region


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def config_of(wl0, wl, world, extra=None):
    """The `config` object of the JSON line: the same keys for the library's arm and the oracle's arm."""
    R = wl.refresh
    full_bytes = wl.batch * wl.seq_len * wl.row_elems * wl.elem_bytes
    cfg = {"workload": wl0.name, "batch_per_gpu": wl.batch, "seq_len": wl.seq_len, "packed_len": wl.packed_len,
           "heads": wl.n_heads, "head_dim": wl.head_dim, "keep": wl.keep, "k_core": wl.budgets[0],
           "k_anchor": wl.budgets[1], "refresh_interval": R,
           "step": f"one refresh cycle: 1 full step + {R - 1} sparse step(s)",
           "tokens_per_step": wl.batch * (wl.seq_len + (R - 1) * wl.packed_len),
           "l2": f"inputs exceed L2: {3 * R * full_bytes / 1e6:.0f} MB of q/k/v per step"
                 if 3 * R * full_bytes > (126 << 20) else "inputs smaller than L2, no flush in the step loop",
           "parallelism": f"sample-sharded x{world}"}
    if extra:
        cfg.update(extra)
    return cfg


# ----------------------------------------------------------------------------------------------------------
# clocks: read-only sampling during the timed region
# ----------------------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, device_index: int, period_s: float = 0.001):
        self.samples, self.stamps, self.reasons, self.max_mhz = [], [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None
        self.period = period_s

    def _loop(self):
        nv = self._nv
        names = {
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.stamps.append(time.perf_counter())
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def stop(self, window=None):
        """window = (t0, t1) in perf_counter time: also reports how many samples fell inside it."""
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        rec = {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
               "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.samples:
            rec["sm_mhz_min"] = int(min(self.samples))
        if window is not None and self.samples:
            inside = [s for s, t in zip(self.samples, self.stamps) if window[0] <= t <= window[1]]
            rec["samples_in_timed_region"] = len(inside)
            if inside:
                rec["sm_mhz_in_timed_region"] = float(np.median(inside))
        return rec


# ----------------------------------------------------------------------------------------------------------
# timing primitives
# ----------------------------------------------------------------------------------------------------------
N_ROT = 4  # rotating input sets for per-stage timing: their footprint exceeds L2 several times over


def graph_of(fn):
    """Capture fn() (which enqueues kernels on the current stream) into a CUDA graph."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()   # warm-up outside capture (first-use attribute calls, tensor maps)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def replay_ms(g, n):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def per_launch_us(fns, min_s):
    """Average device time per launch: the callables (one per rotating input set, so consecutive launches read cold
    data) are captured into one CUDA graph that is replayed back to back between two events for at least `min_s`
    seconds (after as long a run-in), so that the figure is a steady-state one."""
    def all_sets():
        for f in fns:
            f()
    g = graph_of(all_sets)
    est_ms = max(replay_ms(g, 2) / 2, 1e-3)
    reps = int(max(3, min(20000, math.ceil(min_s * 1e3 / est_ms))))
    replay_ms(g, reps)                                  # run-in of the same length
    return replay_ms(g, reps) * 1e3 / (reps * len(fns))


def first_launches_us(fns, n_launches=24):
    """Device time per launch right after an idle gap (clocks at maximum, power cap not yet engaged): median over
    the launches 2 .. n of one back-to-back run."""
    torch.cuda.synchronize()
    time.sleep(0.5)
    for f in fns:
        f()                                             # wake the clocks
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_launches + 1)]
    marks[0].record()
    for i in range(n_launches):
        fns[i % len(fns)]()
        marks[i + 1].record()
    torch.cuda.synchronize()
    t = [marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(n_launches)]
    return float(np.median(t[2:]))


# ----------------------------------------------------------------------------------------------------------
# the swam arm
# ----------------------------------------------------------------------------------------------------------
def measure_workload(wl0, args, rank, local_rank, world, device, peaks, peak_kind, detail):
    """Times one workload.  detail = True: the full stage table, oracle baseline and end-to-end leg (the line's own
    workload); False: cycle, steps, attention stages and end-to-end leg only (the `also` records)."""
    from paper_2609_38984_b200 import swam
    wl = sd.rank_workload(wl0, rank, world)
    R = wl.refresh
    gen = W.Generator(wl)
    host_steps = [gen.next_step() for _ in range(R)]
    tdt = swam.torch_dtype(wl.dtype)
    host_pinned = [{n: torch.from_numpy(x[n]).to(tdt).pin_memory() for n in "qkv"} for x in host_steps]
    dev_steps = [{n: hp[n].to(device, non_blocking=True) for n in "qkv"} for hp in host_pinned]
    ctx = swam.Swam.from_workload(wl)
    out = ctx.empty_full().zero_()
    torch.cuda.synchronize()
    modes = [swam.REFRESH_FULL] + [swam.REUSE] * (R - 1)

    def cycle():
        for x, m in zip(dev_steps, modes):
            ctx.step(x["q"], x["k"], x["v"], m, out)

    # the cycle has a fixed shape (fixed packed length), so it is captured once and replayed
    l0 = ctx.launch_count()
    cycle()
    launches_per_cycle = ctx.launch_count() - l0
    cycle_graph = graph_of(cycle)
    warm = max(args.warmup, 3)
    for _ in range(warm):
        cycle_graph.replay()
    ctx.check()
    est_ms = max(replay_ms(cycle_graph, 3) / 3, 1e-3)

    def timed(preload_s, idle_s):
        """Exactly args.steps cycles between two events, after `idle_s` of idle + the warm-up replays (burst) or after
        `preload_s` of back-to-back replays (steady); max over ranks; clocks sampled throughout."""
        torch.cuda.synchronize()
        if idle_s:
            time.sleep(idle_s)
        sampler = ClockSampler(local_rank).start()
        n_pre = int(math.ceil(preload_s * 1e3 / est_ms)) if preload_s else warm
        for _ in range(n_pre):
            cycle_graph.replay()
        sd.barrier(device)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record()
        for _ in range(args.steps):
            cycle_graph.replay()
        e1.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        clocks = sampler.stop(window=(t0, t1))
        sd.barrier(device)
        ms = sd.max_over_ranks(e0.elapsed_time(e1), device)
        clocks["replays_before_timed_region"] = n_pre
        return ms, clocks

    ms_burst, clocks_burst = timed(0.0, 0.5)
    ms_steady, clocks_steady = timed(args.preload_seconds, 0.0)
    ctx.check()
    tokens_per_cycle = wl.batch * (wl.seq_len + (R - 1) * wl.packed_len)
    value = world * tokens_per_cycle * args.steps / (ms_steady * 1e-3)
    value_burst = world * tokens_per_cycle * args.steps / (ms_burst * 1e-3)

    # end to end: pinned host tensors in, host result out, through the host-buffer entry point
    out_host = torch.empty(out.shape, dtype=tdt).pin_memory()
    ctx.bind_host_io()
    e2e_steps = max(2, min(args.steps, 10))

    def cycle_host():
        for hp, m in zip(host_pinned, modes):
            ctx.step_host(hp["q"], hp["k"], hp["v"], m, out_host)

    cycle_host()
    torch.cuda.synchronize()
    sd.barrier(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        cycle_host()
    ctx.host_join()      # the timed region ends when the last result has arrived in host memory
    e1.record()
    torch.cuda.synchronize()
    sd.barrier(device)
    e2e_ms = sd.max_over_ranks(e0.elapsed_time(e1), device)
    ctx.check()
    full_bytes = out.numel() * out.element_size()
    kv_bytes = full_bytes * wl.kv_heads // wl.n_heads
    e2e = {"value": world * tokens_per_cycle * e2e_steps / (e2e_ms * 1e-3), "unit": "tokens/s",
           # a reuse step brings only the rows its maps retain across PCIe (the library's default for pinned buffers)
           "h2d_bytes_per_step": (full_bytes + 2 * kv_bytes) * (wl.seq_len + (R - 1) * wl.packed_len) // wl.seq_len,
           "d2h_bytes_per_step": full_bytes * R,
           "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps}

    rec = {"value": value, "value_burst": value_burst, "unit": "tokens/s", "ms_per_step": ms_steady / args.steps,
           "ms_per_step_burst": ms_burst / args.steps, "clocks": clocks_steady, "clocks_burst": clocks_burst,
           "e2e": e2e, "gpu_launches": int(launches_per_cycle * args.steps),
           "config": config_of(wl0, wl, world, {
               "timing": f"CUDA-graph replays, CUDA events; value: {args.steps} cycles right after >= {args.preload_seconds:g} s "
                         f"of back-to-back replays (steady state under the power cap); value_burst: {args.steps} cycles "
                         f"after 0.5 s idle and {warm} warm-up cycles",
               "stage_timing": f"per stage: {N_ROT} rotating input sets (each launch reads cold data), launches replayed "
                               f"back to back from a CUDA graph for >= {args.stage_seconds:g} s (attention, steps) or >= "
                               f"{args.stage_seconds / 6:g} s (others) "
                               "after a run-in of the same length, CUDA events around the loop"})}
    if rank != 0:
        return rec

    # per-stage device times through the individual C-ABI calls; every launch of a stage reads one of N_ROT
    # rotating input sets (together several times L2), launches are replayed back to back from a CUDA graph
    lib, P, S = ctx.lib, swam._ptr, swam._stream
    x0, x1 = dev_steps[0], dev_steps[-1]
    rot = [{n: (x0[n] if i == 0 else x1[n] if i == 1 else x0[n].clone()) for n in "qkv"} for i in range(N_ROT)]
    _, lse_act, _ = ctx.cached_scores()
    lse_act = lse_act.clone()
    sel, pm, im = (t.clone() for t in ctx.selection())
    scores = [ctx.score(r["q"], r["k"], lse_act) for r in rot]
    packed = [ctx.pack(r["q"], r["k"], r["v"], pm) for r in rot]
    outs_p = [ctx.sparse_attn(*pk) for pk in packed]
    outs = [out] + [out.clone() for _ in range(N_ROT - 1)]
    eb = wl.elem_bytes
    row = wl.row_elems * eb
    row_kv = wl.kv_heads * wl.head_dim * eb
    B, L, Lp = wl.batch, wl.seq_len, wl.packed_len
    fut = wl.n_frames * wl.n_spatial
    stage_clocks = {}

    long_s, short_s = args.stage_seconds, args.stage_seconds / 6

    def stage(make, min_s=short_s, clock_key=None):
        smp = ClockSampler(local_rank, period_s=0.002).start() if clock_key else None
        us = per_launch_us([make(i) for i in range(N_ROT)], min_s)
        if smp:
            stage_clocks[clock_key] = smp.stop()
        return us

    def dense_call(i):
        return lambda: lib.swam_sparse_attn(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]), L, P(outs[i]), None, S())

    def packed_call(i):
        return lambda: lib.swam_sparse_attn(ctx.ctx, P(packed[i][0]), P(packed[i][1]), P(packed[i][2]), Lp, P(outs_p[i]),
                                            None, S())

    def step_call(mode):
        return lambda i: lambda: lib.swam_step(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]), mode, P(outs[i]), S())

    stage_us = {
        "attn_dense": stage(dense_call, long_s, "attn_dense"),
        "attn_packed": stage(packed_call, long_s, "attn_packed"),
        "full_step": stage(step_call(swam.REFRESH_FULL), long_s, "full_step"),
        "sparse_step": stage(step_call(swam.REUSE), long_s, "sparse_step"),
    }
    if wl.dtype == W.BF16 and wl.head_dim >= 64:
        # the sparse step with the key and value rows gathered inside the attention kernel (one launch, nothing packed)
        ctx.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_FUSED_KV)
        stage_us["sparse_step_kv_gathered_in_kernel"] = stage(step_call(swam.REUSE), long_s)
        ctx.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_FUSED)
    burst_us = {"attn_dense": first_launches_us([dense_call(i) for i in range(N_ROT)]),
                "attn_packed": first_launches_us([packed_call(i) for i in range(N_ROT)])}
    if detail:
        stage_us.update({
            "score": stage(lambda i: lambda: lib.swam_score(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(lse_act), P(scores[i]),
                                                            None, S())),
            "score_with_lse": stage(lambda i: lambda: lib.swam_score(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), None,
                                                                     P(scores[i]), None, S())),
            "select": stage(lambda i: lambda: lib.swam_select(ctx.ctx, P(scores[i]), P(sel), P(pm), P(im), S())),
            "launch_floor": stage(lambda i: lambda: lib.swam_launch_floor(ctx.ctx, S())),
            "pack": stage(lambda i: lambda: lib.swam_pack(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]), P(pm),
                                                          P(packed[i][0]), P(packed[i][1]), P(packed[i][2]), S())),
            "pack_kv": stage(lambda i: lambda: lib.swam_pack(ctx.ctx, None, P(rot[i]["k"]), P(rot[i]["v"]), P(pm),
                                                             None, P(packed[i][1]), P(packed[i][2]), S())),
            "scatter": stage(lambda i: lambda: lib.swam_scatter(ctx.ctx, P(outs_p[i]), P(pm), P(im), P(outs[i]), P(outs[i]),
                                                                S())),
            "light_refresh_step": stage(step_call(swam.REFRESH_LIGHT), long_s / 3),
        })
        # several profiled layers (Eq. 3, Eq. 9, Eq. 11): six layers' score maps and qualities -> core map over the
        # three best layers and anchor map over all, then the selection from the two maps
        n_layers, k_layer = 6, 3
        layer_s = torch.stack([scores[i % N_ROT] for i in range(n_layers)]).contiguous()
        layer_q = torch.rand((n_layers, B, 3), device=device, dtype=torch.float32)
        v_core, v_all, core_layers = ctx.aggregate(layer_s, layer_q, k_layer)
        stage_us["aggregate_6_layers"] = stage(lambda i: lambda: lib.swam_aggregate(
            ctx.ctx, P(layer_s), P(layer_q), n_layers, k_layer, P(v_core), P(v_all), P(core_layers), S()))
        stage_us["select_two_maps"] = stage(lambda i: lambda: lib.swam_select_maps(
            ctx.ctx, P(v_core), P(v_all), P(sel), P(pm), P(im), S()))
        if wl.dtype == W.BF16 and wl.head_dim >= 64:
            # restricted visibility (App. A.2's constraints in the segment-prefix form): observed rows see the observed
            # tokens only, future rows the observed and future ones, action rows everything
            ctx.set_visibility(swam.SEES_OBSERVED, swam.SEES_FUTURE, swam.SEES_ALL)
            stage_us["full_step_segment_visibility"] = stage(step_call(swam.REFRESH_FULL), long_s / 3)
            stage_us["sparse_step_segment_visibility"] = stage(step_call(swam.REUSE), long_s / 3)
            ctx.set_visibility(swam.SEES_ALL, swam.SEES_ALL, swam.SEES_ALL)
    ctx.check()
    algo = {  # algorithmic bytes / flops per launch
        "score": ("hbm", B * (fut * row_kv + wl.n_action * row + fut * 4)),
        "score_with_lse": ("hbm", B * (L * row_kv + wl.n_action * row + fut * 4)),
        "pack": ("hbm", 2 * B * Lp * (row + 2 * row_kv)),
        "pack_kv": ("hbm", 2 * B * Lp * 2 * row_kv),
        "scatter": ("hbm", 2 * B * Lp * row),
        "attn_packed": ("tensor", 4.0 * B * wl.n_heads * Lp * Lp * wl.head_dim),
        "attn_dense": ("tensor", 4.0 * B * wl.n_heads * L * L * wl.head_dim),
    }
    stages = {}
    for name, (bound, work) in algo.items():
        if name not in stage_us:
            continue
        us = stage_us[name]
        if bound == "hbm":
            ach = work / (us * 1e-6) / 1e9
            stages[name] = {"us": round(us, 2), "bound": "hbm", "bytes": int(work), "achieved_gbs": round(ach, 1),
                            "frac": round(ach / peaks["hbm_gbs"], 4)}
        else:
            ach = work / (us * 1e-6) / 1e12
            ach_b = work / (burst_us[name] * 1e-6) / 1e12
            stages[name] = {"us": round(us, 2), "bound": "tensor", "flops": work, "achieved_tflops": round(ach, 1),
                            "frac_of_sustained_peak": round(ach / peaks["bf16_tflops_sustained"], 4),
                            "us_burst": round(burst_us[name], 2), "achieved_tflops_burst": round(ach_b, 1),
                            "frac": round(ach_b / peaks["bf16_tflops"], 4),
                            "regime": "us: steady back-to-back loop (sustained peak); us_burst: first launches after "
                                      "an idle gap (burst peak, which `frac` refers to)"}
    if "select" in stage_us:
        # selection reads at most a few hundred KB: it is bound by launch and dependent-pass latency, so it is
        # reported against the launch floor (an empty kernel in the same harness), not against memory bandwidth
        stages["select"] = {"us": round(stage_us["select"], 2), "bound": "latency",
                            "launch_floor_us": round(stage_us["launch_floor"], 2),
                            "ratio_to_launch_floor": round(stage_us["select"] / stage_us["launch_floor"], 2),
                            "bytes": int(B * (fut * 4 + (wl.n_frames * wl.k_keep + Lp + L) * 4))}
    if "aggregate_6_layers" in stage_us:
        agg_bytes = B * fut * 4 * (6 + 2)
        stages["aggregate_6_layers"] = {"us": round(stage_us["aggregate_6_layers"], 2), "bound": "latency", "bytes": int(agg_bytes),
                                        "ratio_to_launch_floor": round(stage_us["aggregate_6_layers"] / stage_us["launch_floor"], 2)}
        stages["select_two_maps"] = {"us": round(stage_us["select_two_maps"], 2), "bound": "latency",
                                     "ratio_to_launch_floor": round(stage_us["select_two_maps"] / stage_us["launch_floor"], 2)}
    for name in ("full_step", "sparse_step", "sparse_step_kv_gathered_in_kernel", "light_refresh_step",
                 "full_step_segment_visibility", "sparse_step_segment_visibility"):
        if name in stage_us:
            stages[name] = {"us": round(stage_us[name], 2)}

    # dominant kernel: the joint-attention kernel (dense launch of the full step + packed launch of the sparse steps),
    # in the regime `value` is quoted in (steady state -> sustained peak); the burst figures stand beside it
    att_flops = algo["attn_dense"][1] + (R - 1) * algo["attn_packed"][1]
    att_us = stage_us["attn_dense"] + (R - 1) * stage_us["attn_packed"]
    att_us_b = burst_us["attn_dense"] + (R - 1) * burst_us["attn_packed"]
    achieved = att_flops / (att_us * 1e-6) / 1e12
    achieved_b = att_flops / (att_us_b * 1e-6) / 1e12
    if wl.dtype == W.BF16:
        roofline = {"kernel": "joint attention (dense + packed launches of one cycle)", "bound": "tensor",
                    "achieved": round(achieved, 2), "peak": round(peaks["bf16_tflops_sustained"], 1), "unit": "TFLOP/s",
                    "frac": round(achieved / peaks["bf16_tflops_sustained"], 4),
                    "peak_source": f"{peak_kind} (sustained bf16 GEMM figure: the stage loops, like `value`, run in the "
                                   "steady state under the power cap)",
                    "burst": {"achieved": round(achieved_b, 2), "peak": round(peaks["bf16_tflops"], 1),
                              "frac": round(achieved_b / peaks["bf16_tflops"], 4),
                              "peak_source": f"{peak_kind} (burst bf16 GEMM figure; launches timed right after an idle gap)"},
                    "traffic": DOMINANT_KERNEL_DRAM_BYTES.get(wl0.name)}
        # the exponential unit: one ex2 per score element = per 4 * D flop of the two products; at head dim 64 it, not
        # the tensor pipe, is the nearer ceiling
        clk = (stage_clocks.get("attn_dense", {}).get("sm_mhz") or clocks_steady.get("sm_mhz") or 1965.0) * 1e6
        ex2_peak = EX2_PER_CLK_PER_SM * N_SMS * clk * 4 * wl.head_dim / 1e12
        roofline["exp2"] = {"bound": "exp2", "achieved": round(achieved, 2), "peak": round(ex2_peak, 1), "unit": "TFLOP/s",
                            "frac": round(achieved / ex2_peak, 4),
                            "peak_source": f"derived: {EX2_PER_CLK_PER_SM} ex2/clk/SM x {N_SMS} SMs x {clk / 1e6:.0f} MHz "
                                           f"(median SM clock sampled during the dense-attention loop) x 4 x {wl.head_dim} "
                                           "flop per exponential; one exponential in eight runs on the FMA pipes instead"}
    else:
        # fp32 tensors run on the FMA pipes: peak = 148 SMs x 128 FP32 lanes x 2 flop x 1.965 GHz (nominal unit counts
        # and the maximum SM clock); the measured tensor peak only applies to bf16
        peak = N_SMS * 128 * 2 * 1.965e9 / 1e12
        roofline = {"kernel": "joint attention (dense + packed launches of one cycle)", "bound": "alu",
                    "achieved": round(achieved, 2), "peak": round(peak, 1), "unit": "TFLOP/s",
                    "frac": round(achieved / peak, 4), "peak_source": "derived: 148 SMs x 128 lanes x 2 x 1.965 GHz",
                    "traffic": None}
    rec.update({"sparse_step_us": stages["sparse_step"]["us"], "full_step_us": stages["full_step"]["us"],
                "roofline": roofline, "stages": stages, "stage_clocks": stage_clocks})
    if detail:
        rec["cpu_baseline"] = cpu_baseline(wl, host_steps, budget_s=args.cpu_seconds)
    del ctx, out, rot, packed, outs_p, outs, dev_steps, host_pinned
    torch.cuda.empty_cache()
    return rec


def bench_swam(args):
    _, local_rank, _ = sd.env_rank()
    torch.cuda.set_device(local_rank)            # before the process group, so NCCL binds this rank to its own GPU
    device = torch.device("cuda", local_rank)
    rank, local_rank, world = sd.init("nccl")
    peaks, peak_kind = load_peaks()
    wl0 = W.WORKLOADS[args.workload]
    rec = measure_workload(wl0, args, rank, local_rank, world, device, peaks, peak_kind, detail=True)
    line = None
    if rank == 0:
        line = {"metric": "packed_tokens_per_s", "value": rec.pop("value"), "unit": rec.pop("unit"), "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": rec.pop("ms_per_step"),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if wl0.dtype == W.BF16 else "f32", "data": "synthetic", "impl": "swam"}
        line.update(rec)
        # the other benchmark shapes, same measurement (one GPU only: every rank of a multi-GPU run has its own batch
        # of the line's workload and nothing else)
        if world == 1 and args.also:
            line["also"] = {}
            for name in args.also.split(","):
                if name and name != wl0.name:
                    a = measure_workload(W.WORKLOADS[name], args, rank, local_rank, world, device, peaks, peak_kind,
                                         detail=False)
                    line["also"][name] = a
    sd.barrier(device)
    sd.finalize()
    if line is not None:
        print(json.dumps(line))


# ----------------------------------------------------------------------------------------------------------
# the oracle on the host cores, on a bounded sample of the same workload
# ----------------------------------------------------------------------------------------------------------
def oracle_cycle_seconds(wl, host_steps, budget_s, all_rows=False):
    """Runs the oracle's refresh cycle with the attention restricted to a sample of query rows sized for about
    `budget_s` seconds (all_rows: every row), and scales the attention part to all rows.  Returns (seconds per
    full cycle, description, measured seconds, attention rows processed)."""
    from oracle import reference as ora
    kc, ks = wl.budgets
    R = wl.refresh
    x0 = host_steps[0]
    rng = np.random.default_rng(0)
    n_all_d, n_all_p = wl.batch * wl.seq_len, wl.batch * wl.packed_len
    if all_rows:
        n_dense, n_packed = n_all_d, n_all_p
        rows_d = np.stack(np.meshgrid(np.arange(wl.batch), np.arange(wl.seq_len), indexing="ij"), -1).reshape(-1, 2)
        rows_p = np.stack(np.meshgrid(np.arange(wl.batch), np.arange(wl.packed_len), indexing="ij"), -1).reshape(-1, 2)
    else:
        # calibrate on 2 rows
        t0 = time.perf_counter()
        ora.attention_rows(x0["q"], x0["k"], x0["v"], np.array([[0, 0], [0, wl.seq_len - 1]]))
        per_row_dense = (time.perf_counter() - t0) / 2
        per_row_packed = per_row_dense * wl.packed_len / wl.seq_len
        share = budget_s / (per_row_dense + (R - 1) * per_row_packed)
        n_dense = int(max(2, min(n_all_d, share)))
        n_packed = int(max(2, min(n_all_p, share)))
        rows_d = np.stack([rng.integers(0, wl.batch, n_dense), rng.integers(0, wl.seq_len, n_dense)], -1)
        rows_p = np.stack([rng.integers(0, wl.batch, n_packed), rng.integers(0, wl.packed_len, n_packed)], -1)
    t0 = time.perf_counter()
    st = ora.StepState()
    ta = time.perf_counter()
    ora.attention_rows(x0["q"], x0["k"], x0["v"], rows_d)
    t_dense_rows = time.perf_counter() - ta
    tb = time.perf_counter()
    lse = ora.action_lse(x0["q"], x0["k"], wl.n_action)
    s = ora.score(x0["q"], x0["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse).astype(np.float32)
    st.sel = ora.select(s, kc, ks)
    st.pack_map, st.inv_map = ora.maps(st.sel["sel_idx"], wl.n_obs, wl.n_spatial, wl.n_action)
    t_sel = time.perf_counter() - tb
    t_sparse_rows, t_pack = 0.0, 0.0
    for x in host_steps[1:R]:
        tc = time.perf_counter()
        qp, kp, vp = ora.pack(x["q"], st.pack_map), ora.pack(x["k"], st.pack_map), ora.pack(x["v"], st.pack_map)
        t_pack += time.perf_counter() - tc
        tc = time.perf_counter()
        ora.attention_rows(qp, kp, vp, rows_p)
        t_sparse_rows += time.perf_counter() - tc
    measured = time.perf_counter() - t0
    est = (t_dense_rows * (n_all_d / n_dense) + t_sel + t_pack + t_sparse_rows * (n_all_p / n_packed))
    desc = (f"oracle refresh cycle with attention on {n_dense} of {n_all_d} dense rows and {n_packed} of "
            f"{n_all_p} packed rows per sparse step (all heads), score/select/maps/pack in full; "
            f"attention time scaled to all rows")
    return est, desc, measured, n_dense + (R - 1) * n_packed


_VALIDATION = None


def extrapolation_check():
    """Row sampling validated once where the oracle finishes in seconds: the single-view shape timed on every row
    against the estimate from a one-second sample."""
    global _VALIDATION
    if _VALIDATION is None:
        wl = W.WORKLOADS["single_view"]
        gen = W.Generator(wl)
        hs = [gen.next_step() for _ in range(wl.refresh)]
        est, _, _, _ = oracle_cycle_seconds(wl, hs, 1.0)
        full, _, _, _ = oracle_cycle_seconds(wl, hs, 0.0, all_rows=True)
        _VALIDATION = {"workload": wl.name, "measured_all_rows_s": round(full, 3), "extrapolated_from_sample_s": round(est, 3),
                       "ratio": round(est / full, 3)}
    return _VALIDATION


def cpu_baseline(wl, host_steps, budget_s):
    from oracle import reference as ora
    est, desc, measured, _ = oracle_cycle_seconds(wl, host_steps, budget_s)
    tokens = wl.batch * (wl.seq_len + (wl.refresh - 1) * wl.packed_len)
    return {"value": tokens / est, "unit": "tokens/s", "cores": ora.threads(), "kind": "oracle", "sample": desc,
            "measured_s": round(measured, 2), "est_s_per_step": round(est, 2), "sampling_check": extrapolation_check()}


def bench_reference(args):
    """The oracle as it stands on the host cores: --warmup untimed and --steps timed steps, each one refresh cycle on a
    bounded sample of the workload (attention on a seeded sample of query rows, everything else in full), sized so that
    the whole run takes about --reference-seconds."""
    rank, _, world = sd.env_rank()
    if rank != 0:
        return
    from oracle import reference as ora
    wl = W.WORKLOADS[args.workload]
    gen = W.Generator(wl)
    host_steps = [gen.next_step() for _ in range(wl.refresh)]
    steps, warm = max(1, args.steps), max(0, args.warmup)
    per = max(0.2, args.reference_seconds / (steps + warm))
    for _ in range(warm):
        oracle_cycle_seconds(wl, host_steps, per)
    ests, walls, desc = [], [], ""
    t_all = time.perf_counter()
    for _ in range(steps):
        t0 = time.perf_counter()
        est, desc, _, _ = oracle_cycle_seconds(wl, host_steps, per)
        walls.append(time.perf_counter() - t0)
        ests.append(est)
    wall = time.perf_counter() - t_all
    est = float(np.mean(ests))
    tokens = wl.batch * (wl.seq_len + (wl.refresh - 1) * wl.packed_len)
    value = tokens / est
    print(json.dumps({
        "impl": "reference", "metric": "packed_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": wall * 1e3 / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, wl, 1, {
            "timing": f"{steps} timed steps after {warm} untimed ones, wall clock; each step is the oracle's refresh cycle on "
                      "a bounded sample (see cpu_baseline.sample); ms_per_step is the measured time of such a step, value "
                      "the workload's tokens per cycle over the cycle time scaled to all rows (est_s_per_step)",
            "stage_timing": "none"}),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": ora.threads(), "kind": "oracle", "sample": desc,
                         "est_s_per_step": round(est, 2), "sampling_check": extrapolation_check()},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="larger_imagination", choices=sorted(W.WORKLOADS))
    ap.add_argument("--also", default="multi_view,single_view",
                    help="further workloads measured the same way and reported under `also` (one GPU only); '' = none")
    ap.add_argument("--impl", default="swam", choices=["swam", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="host-core budget of the oracle baseline")
    ap.add_argument("--preload-seconds", type=float, default=STEADY_PRELOAD_S,
                    help="back-to-back replays before the steady-state timed region (shorten only for profiler runs)")
    ap.add_argument("--stage-seconds", type=float, default=0.3,
                    help="length of the per-stage timing loops of the attention launches and steps (others: a sixth)")
    ap.add_argument("--reference-seconds", type=float, default=120.0,
                    help="host-core budget of the whole --impl reference run (all warm-up and timed steps)")
    args = ap.parse_args()
    if args.impl == "reference":
        bench_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    bench_swam(args)


if __name__ == "__main__":
    main()
