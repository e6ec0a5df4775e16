#!/usr/bin/env python
"""Benchmark of the sparse denoising step on B200.

A timed "step" is one refresh cycle of the workload's schedule (refresh interval R, default 2): one full step
(dense joint attention + action-to-future scoring + selection and maps) followed by R-1 sparse steps (pack,
packed joint attention, scatter) that reuse the selection.  `value` is the number of tokens that went through the
joint attention per second, B * (L + (R-1) L') per cycle, summed over ranks.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl swam|reference]

For N > 1 launch through torch.distributed.run (one rank per GPU); a plain `--gpus N` invocation re-launches
itself that way.  Every rank runs its own batch of samples (weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
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


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------------------------------------
# clocks: read-only sampling during the timed region
# ----------------------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, device_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
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

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------------------------------------
# the swam arm
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


def per_launch_us(fns, reps):
    """Average device time per launch: the callables (one per rotating input set, so consecutive launches read cold
    data) are captured into one CUDA graph that is replayed `reps` times between two events."""
    def all_sets():
        for f in fns:
            f()
    g = graph_of(all_sets)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * len(fns))


def power_profile_us(fns, n_launches=160):
    """Device time per launch at the start and at the end of one back-to-back run of `n_launches` launches (rotating
    input sets), after a short idle: the difference shows how much of the steady-state time is the power cap."""
    torch.cuda.synchronize()
    time.sleep(0.5)
    for f in fns:
        f()                                        # wake the clocks
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_launches + 1)]
    marks[0].record()
    for i in range(n_launches):
        fns[i % len(fns)]()
        marks[i + 1].record()
    torch.cuda.synchronize()
    t = [marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(n_launches)]
    k = max(4, n_launches // 8)
    return float(np.median(t[2:2 + k])), float(np.median(t[-k:]))


def bench_swam(args):
    from paper_2609_38984_b200 import swam
    _, local_rank, _ = sd.env_rank()
    torch.cuda.set_device(local_rank)            # before the process group, so NCCL binds this rank to its own GPU
    device = torch.device("cuda", local_rank)
    rank, local_rank, world = sd.init("nccl")
    wl0 = W.WORKLOADS[args.workload]
    wl = sd.rank_workload(wl0, rank, world)
    R = wl.refresh
    peaks, peak_kind = load_peaks()

    # inputs: one tensor set per denoising step of the cycle, resident in HBM before timing
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
    for _ in range(max(args.warmup, 3)):
        cycle_graph.replay()
    ctx.check()

    sampler = ClockSampler(local_rank)
    sd.barrier(device)
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        cycle_graph.replay()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    sd.barrier(device)
    ms_local = e0.elapsed_time(e1)
    launches = launches_per_cycle * args.steps
    ctx.check()
    ms_total = sd.max_over_ranks(ms_local, device)
    tokens_per_cycle = wl.batch * (wl.seq_len + (R - 1) * wl.packed_len)
    value = world * tokens_per_cycle * args.steps / (ms_total * 1e-3)

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
    e2e = {"value": world * tokens_per_cycle * e2e_steps / (e2e_ms * 1e-3), "unit": "tokens/s",
           "h2d_bytes_per_step": 3 * full_bytes * R, "d2h_bytes_per_step": full_bytes * R,
           "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps}

    line = None
    if rank == 0:
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
        B, L, Lp = wl.batch, wl.seq_len, wl.packed_len
        fut = wl.n_frames * wl.n_spatial
        reps = max(3, min(args.steps, 20))

        stage_clocks = {}

        def stage(make, clock_key=None):
            smp = ClockSampler(local_rank, period_s=0.005) if clock_key else None
            if smp:
                smp.start()
            us = per_launch_us([make(i) for i in range(N_ROT)], reps)
            if smp:
                stage_clocks[clock_key] = smp.stop()
            return us

        stage_us = {
            "attn_dense": stage(lambda i: lambda: lib.swam_sparse_attn(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]), L,
                                                                       P(outs[i]), None, S()), "attn_dense"),
            "score": stage(lambda i: lambda: lib.swam_score(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(lse_act), P(scores[i]),
                                                            None, S())),
            "score_with_lse": stage(lambda i: lambda: lib.swam_score(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), None,
                                                                     P(scores[i]), None, S())),
            "select": stage(lambda i: lambda: lib.swam_select(ctx.ctx, P(scores[i]), P(sel), P(pm), P(im), S())),
            "pack": stage(lambda i: lambda: lib.swam_pack(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]), P(pm),
                                                          P(packed[i][0]), P(packed[i][1]), P(packed[i][2]), S())),
            "attn_packed": stage(lambda i: lambda: lib.swam_sparse_attn(ctx.ctx, P(packed[i][0]), P(packed[i][1]),
                                                                        P(packed[i][2]), Lp, P(outs_p[i]), None, S())),
            "scatter": stage(lambda i: lambda: lib.swam_scatter(ctx.ctx, P(outs_p[i]), P(pm), P(im), P(outs[i]), P(outs[i]),
                                                                S())),
            "full_step": stage(lambda i: lambda: lib.swam_step(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]),
                                                               swam.REFRESH_FULL, P(outs[i]), S())),
            "sparse_step": stage(lambda i: lambda: lib.swam_step(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]),
                                                                 swam.REUSE, P(outs[i]), S())),
            "light_refresh_step": stage(lambda i: lambda: lib.swam_step(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]),
                                                                        P(rot[i]["v"]), swam.REFRESH_LIGHT, P(outs[i]), S())),
        }
        dense_fns = [(lambda i: lambda: lib.swam_sparse_attn(ctx.ctx, P(rot[i]["q"]), P(rot[i]["k"]), P(rot[i]["v"]), L,
                                                             P(outs[i]), None, S()))(i) for i in range(N_ROT)]
        dense_first_us, dense_late_us = power_profile_us(dense_fns)
        ctx.check()
        algo = {  # algorithmic bytes / flops per launch
            "score": ("hbm", B * (fut * row + wl.n_action * row + wl.n_frames * wl.n_spatial * 4)),
            "score_with_lse": ("hbm", B * (L * row + wl.n_action * row + wl.n_frames * wl.n_spatial * 4)),
            "select": ("hbm", B * (wl.n_frames * wl.n_spatial * 4 + (wl.n_frames * wl.k_keep + Lp + L) * 4)),
            "pack": ("hbm", 2 * 3 * B * Lp * row),
            "scatter": ("hbm", 2 * B * Lp * row),
            "attn_packed": ("tensor", 4.0 * B * wl.n_heads * Lp * Lp * wl.head_dim),
            "attn_dense": ("tensor", 4.0 * B * wl.n_heads * L * L * wl.head_dim),
        }
        stages = {}
        for name, (bound, work) in algo.items():
            us = stage_us[name]
            if bound == "hbm":
                ach = work / (us * 1e-6) / 1e9
                stages[name] = {"us": round(us, 2), "bound": "hbm", "bytes": int(work), "achieved_gbs": round(ach, 1),
                                "frac": round(ach / peaks["hbm_gbs"], 4)}
            else:
                ach = work / (us * 1e-6) / 1e12
                stages[name] = {"us": round(us, 2), "bound": "tensor", "flops": work, "achieved_tflops": round(ach, 1),
                                "frac": round(ach / peaks["bf16_tflops"], 4)}
        for name in ("full_step", "sparse_step", "light_refresh_step"):
            stages[name] = {"us": round(stage_us[name], 2)}
        # the dense launch right after an idle gap and after ~0.15 s of back-to-back launches (power cap engaged)
        stages["attn_dense"]["us_first_launches_after_idle"] = round(dense_first_us, 2)
        stages["attn_dense"]["us_after_160_back_to_back"] = round(dense_late_us, 2)
        # dominant kernel: the joint-attention kernel (dense launch of the full step + packed launch of the sparse steps)
        att_flops = algo["attn_dense"][1] + (R - 1) * algo["attn_packed"][1]
        att_us = stage_us["attn_dense"] + (R - 1) * stage_us["attn_packed"]
        achieved = att_flops / (att_us * 1e-6) / 1e12
        # fp32 tensors run on the FMA pipes: peak = 148 SMs x 128 FP32 lanes x 2 flop x 1.965 GHz (nominal unit counts
        # and the maximum SM clock); the measured tensor peak only applies to bf16
        if wl.dtype == W.BF16:
            bound, peak, src = "tensor", peaks["bf16_tflops"], f"{peak_kind} (burst)"
        else:
            bound, peak, src = "alu", 148 * 128 * 2 * 1.965e9 / 1e12, "derived: 148 SMs x 128 lanes x 2 x 1.965 GHz"
        roofline = {"kernel": "joint attention (dense + packed launches of one cycle)", "bound": bound,
                    "achieved": round(achieved, 2), "peak": round(peak, 1), "unit": "TFLOP/s",
                    "frac": round(achieved / peak, 4), "peak_source": src,
                    "traffic": DOMINANT_KERNEL_DRAM_BYTES.get(wl0.name)}
        if wl.dtype == W.BF16:
            # the stage loop runs long enough for the power cap to engage, which is the regime the sustained GEMM
            # figure was measured in; the headline fraction above stays on the (larger) burst figure
            roofline["frac_of_sustained_peak"] = round(achieved / peaks["bf16_tflops_sustained"], 4)
            roofline["sustained_peak"] = peaks["bf16_tflops_sustained"]
        cpu = cpu_baseline(wl, host_steps, budget_s=args.cpu_seconds)
        line = {
            "metric": "packed_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.dtype == W.BF16 else "f32", "data": "synthetic",
            "config": {"workload": wl0.name, "batch_per_gpu": wl.batch, "seq_len": wl.seq_len, "packed_len": wl.packed_len,
                       "heads": wl.n_heads, "head_dim": wl.head_dim, "keep": wl.keep, "k_core": wl.budgets[0],
                       "k_anchor": wl.budgets[1], "refresh_interval": R,
                       "step": f"one refresh cycle: 1 full step + {R - 1} sparse step(s), replayed from a CUDA graph",
                       "tokens_per_step": tokens_per_cycle,
                       "l2": f"inputs exceed L2: {3 * R * full_bytes / 1e6:.0f} MB of q/k/v per step"
                             if 3 * R * full_bytes > (126 << 20) else "inputs smaller than L2, no flush in the step loop",
                       "stage_timing": f"per stage: {N_ROT} rotating input sets (each launch reads cold data), launches "
                                       "replayed back to back from a CUDA graph, CUDA events around the loop",
                       "parallelism": f"sample-sharded x{world}"},
            "sparse_step_us": stages["sparse_step"]["us"], "full_step_us": stages["full_step"]["us"],
            "roofline": roofline, "stages": stages, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks, "stage_clocks": stage_clocks, "impl": "swam",
        }
    sd.barrier(device)
    sd.finalize()
    if line is not None:
        print(json.dumps(line))


# ----------------------------------------------------------------------------------------------------------
# the oracle on the host cores, on a bounded sample of the same workload
# ----------------------------------------------------------------------------------------------------------
def oracle_cycle_seconds(wl, host_steps, budget_s):
    """Runs the oracle's refresh cycle with the attention restricted to a sample of query rows sized for about
    `budget_s` seconds, and extrapolates the attention part to all rows.  Returns (seconds per full cycle,
    description, measured seconds)."""
    from oracle import reference as ora
    kc, ks = wl.budgets
    R = wl.refresh
    x0 = host_steps[0]
    rng = np.random.default_rng(0)
    # calibrate on 2 rows
    t0 = time.perf_counter()
    ora.attention_rows(x0["q"], x0["k"], x0["v"], np.array([[0, 0], [0, wl.seq_len - 1]]))
    per_row_dense = (time.perf_counter() - t0) / 2
    per_row_packed = per_row_dense * wl.packed_len / wl.seq_len
    share = budget_s / (per_row_dense + (R - 1) * per_row_packed)
    n_dense = int(max(2, min(wl.batch * wl.seq_len, share)))
    n_packed = int(max(2, min(wl.batch * wl.packed_len, share)))
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
    est = (t_dense_rows * (wl.batch * wl.seq_len / n_dense) + t_sel + t_pack +
           t_sparse_rows * (wl.batch * wl.packed_len / n_packed))
    desc = (f"oracle refresh cycle with attention on {n_dense} of {wl.batch * wl.seq_len} dense rows and {n_packed} of "
            f"{wl.batch * wl.packed_len} packed rows per sparse step (all heads), score/select/maps/pack in full; "
            f"attention time scaled to all rows")
    return est, desc, measured


def cpu_baseline(wl, host_steps, budget_s):
    from oracle import reference as ora
    est, desc, measured = oracle_cycle_seconds(wl, host_steps, budget_s)
    tokens = wl.batch * (wl.seq_len + (wl.refresh - 1) * wl.packed_len)
    return {"value": tokens / est, "unit": "tokens/s", "cores": ora.threads(), "kind": "oracle", "sample": desc,
            "measured_s": round(measured, 2), "est_s_per_step": round(est, 2)}


def bench_reference(args):
    rank, _, world = sd.env_rank()
    if rank != 0:
        return
    from oracle import reference as ora
    wl = W.WORKLOADS[args.workload]
    gen = W.Generator(wl)
    host_steps = [gen.next_step() for _ in range(wl.refresh)]
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    per = max(2.0, args.cpu_seconds / (steps + warm))
    for _ in range(warm):
        oracle_cycle_seconds(wl, host_steps, per)
    ests, desc = [], ""
    for _ in range(steps):
        est, desc, _ = oracle_cycle_seconds(wl, host_steps, per)
        ests.append(est)
    est = float(np.mean(ests))
    tokens = wl.batch * (wl.seq_len + (wl.refresh - 1) * wl.packed_len)
    value = tokens / est
    print(json.dumps({
        "impl": "reference", "metric": "packed_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": est * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch_per_gpu": wl.batch, "seq_len": wl.seq_len, "packed_len": wl.packed_len,
                   "heads": wl.n_heads, "head_dim": wl.head_dim, "keep": wl.keep, "refresh_interval": wl.refresh,
                   "step": f"one refresh cycle: 1 full step + {wl.refresh - 1} sparse step(s)", "tokens_per_step": tokens},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": ora.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="larger_imagination", choices=sorted(W.WORKLOADS))
    ap.add_argument("--impl", default="swam", choices=["swam", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="host-core budget of the oracle baseline")
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
