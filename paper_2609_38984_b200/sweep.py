"""Keep-ratio x refresh-interval sweep at the larger-imagination shape (seed 4), and the paper's ablations on the shapes
of its Table 5: selection strategy (combined, core only, stable anchors only, random; Sec. 5.4), retained tokens per
frame (256 / 184 / 112 of 360; Sec. 5.4) and refresh schedule (first step only, or every R-th step; App. C.2).

For each (keep, R) the workload's 10 denoising steps run through swam_step on one GPU; every stage is also timed
on its own through the individual C-ABI calls.  Reported per configuration: the latency split over score, select,
pack, attention (dense and packed) and scatter, the step latencies (eager, one launch sequence per step) and the device
time of the whole schedule replayed from a CUDA graph, packed tokens/s, the overlap of consecutive
steps' selections (IoU of retained sets and the Eq. 13 overlap of the normalised score maps, from a diagnostic
score + select at every step), and how far the sparse output is from the dense one (relative L2; a reported
number, not a pass/fail: the paper gives no figure for it).

  python -m paper_2609_38984_b200.sweep [--keeps 0.1,0.3] [--refresh 1,2,4] [--steps 10] > sweep.jsonl
  python -m paper_2609_38984_b200.sweep --summarise sweep.jsonl        # the records as a text table (no GPU needed)
  python -m paper_2609_38984_b200.sweep --shape cosmos3_nano --variants combined,core_only,stable_only,random \
         --budgets 256,184,112 --refresh first,1,2
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import swam
from . import workloads as W


def _event_us(fn, reps=5):
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b) * 1e3)
    return float(np.median(ts))


def _graph_us(fn, launches=8, reps=3):
    """Average device time of one fn() when `launches` of them are replayed back to back from a CUDA graph."""
    fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(launches):
            fn()
    g.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        g.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / (launches * reps)


def run_config(wl: W.Workload, refresh: int, n_steps: int, dev_steps, dense_outs, variant: str = "combined") -> dict:
    """`wl` carries the budgets (see workloads.variant_workload); refresh = n_steps runs only the first step in full."""
    keep = wl.keep
    ctx = swam.Swam.from_workload(wl)
    diag = swam.Swam.from_workload(wl)          # diagnostic scoring/selection at every step
    out = ctx.empty_full().zero_()
    sched = W.refresh_schedule(n_steps, refresh)
    # untimed first use (module load, lazily created descriptors), then the whole schedule replayed from a CUDA graph:
    # the device time of the action chunk without host launch overhead, which dominates eager timing of small shapes
    ctx.step(dev_steps[0]["q"], dev_steps[0]["k"], dev_steps[0]["v"], swam.REFRESH_FULL, out)
    ctx.step(dev_steps[0]["q"], dev_steps[0]["k"], dev_steps[0]["v"], swam.REUSE, out)
    ctx.check()
    graph_us = None
    if variant != "random":                      # the random variant installs its keys from the host between steps
        def whole_schedule():
            for t, x in enumerate(dev_steps):
                ctx.step(x["q"], x["k"], x["v"], swam.REFRESH_FULL if sched[t] else swam.REUSE, out)
        graph_us = _graph_us(whole_schedule, launches=1, reps=5)

    step_us, rel_l2, ious, overlaps = [], [], [], []
    prev_sel, prev_scores = None, None
    for t, x in enumerate(dev_steps):
        mode = swam.REFRESH_FULL if sched[t] else swam.REUSE
        step_us.append(_event_us(lambda: ctx.step(x["q"], x["k"], x["v"], mode, out), reps=1))
        if sched[t] and variant == "random":
            # random selection: the same budget per frame, ranked by keys that carry no information
            keys = torch.from_numpy(W.random_scores(wl.seed * 1000 + t, wl.batch, wl.n_frames, wl.n_spatial)).cuda()
            ctx.set_selection(*ctx.select(keys))
        ctx.check()
        d = dense_outs[t].float()
        rel_l2.append(float((out.float() - d).norm() / d.norm()))
        s = diag.score(x["q"], x["k"])
        sel, _, _ = diag.select(s)
        sel_np, s_np = sel.cpu().numpy(), s.cpu().numpy().astype(np.float64)
        if prev_sel is not None:
            inter = [len(np.intersect1d(a, b)) for a, b in zip(prev_sel.reshape(-1, sel_np.shape[-1]),
                                                               sel_np.reshape(-1, sel_np.shape[-1]))]
            k = sel_np.shape[-1]
            ious.append(float(np.mean([i / (2 * k - i) for i in inter])))
            p = prev_scores / prev_scores.sum(-1, keepdims=True)
            q = s_np / s_np.sum(-1, keepdims=True)
            overlaps.append(float(np.minimum(p, q).sum(-1).mean()))      # Eq. 13 per (sample, frame)
        prev_sel, prev_scores = sel_np, s_np
    # stage split on the last step's inputs with the cached selection
    x = dev_steps[-1]
    _, lse_act, _ = ctx.cached_scores()
    sel, pm, im = ctx.selection()
    scores = ctx.score(x["q"], x["k"], lse_act)
    qp, kp, vp = ctx.pack(x["q"], x["k"], x["v"], pm)
    op = ctx.sparse_attn(qp, kp, vp)
    lib, P, S = ctx.lib, swam._ptr, swam._stream
    split = {
        "score": _graph_us(lambda: lib.swam_score(ctx.ctx, P(x["q"]), P(x["k"]), P(lse_act), P(scores), None, S())),
        "select": _graph_us(lambda: lib.swam_select(ctx.ctx, P(scores), P(sel), P(pm), P(im), S())),
        "pack": _graph_us(lambda: lib.swam_pack(ctx.ctx, P(x["q"]), P(x["k"]), P(x["v"]), P(pm), P(qp), P(kp), P(vp), S())),
        "attn_packed": _graph_us(lambda: lib.swam_sparse_attn(ctx.ctx, P(qp), P(kp), P(vp), wl.packed_len, P(op), None, S())),
        "scatter": _graph_us(lambda: lib.swam_scatter(ctx.ctx, P(op), P(pm), P(im), P(out), P(out), S())),
        "attn_dense": _graph_us(lambda: lib.swam_sparse_attn(ctx.ctx, P(x["q"]), P(x["k"]), P(x["v"]), wl.seq_len, P(out), None, S()),
                                launches=4),
    }
    ctx.check()
    full = [u for u, f in zip(step_us, sched) if f]
    sparse = [u for u, f in zip(step_us, sched) if not f]
    total_us = float(np.sum(step_us))
    tokens = wl.batch * sum(wl.seq_len if f else wl.packed_len for f in sched)
    return {
        "shape": wl.name, "variant": variant, "keep": round(keep, 4), "refresh": refresh, "k_core": wl.budgets[0], "k_anchor": wl.budgets[1], "packed_len": wl.packed_len,
        "steps": n_steps, "full_steps": len(full), "stage_us": {k: round(v, 2) for k, v in split.items()},
        "full_step_us": round(float(np.median(full)), 1), "sparse_step_us": round(float(np.median(sparse)), 1) if sparse else None,
        "schedule_us": round(total_us, 1),
        "schedule_graph_us": None if graph_us is None else round(graph_us, 1),
        "tokens_per_s": tokens / ((graph_us if graph_us is not None else total_us) * 1e-6),
        "iou_consecutive_steps": None if variant == "random" else round(float(np.mean(ious)), 4),
        "overlap_eq13_consecutive_steps": round(float(np.mean(overlaps)), 4),
        "rel_l2_vs_dense_per_step": [round(v, 4) for v in rel_l2],
    }


def summarise(path: str) -> str:
    """The JSON lines of a sweep run as a fixed-width text table (one row per configuration)."""
    rows = [json.loads(ln) for ln in open(path) if ln.startswith("{")]
    head = ("shape", "variant", "keep", "R", "K_c+K_s", "L'", "score", "select", "pack", "attn_p", "scatter", "attn_d",
            "full", "sparse", "sched(graph)", "Mtok/s", "IoU", "Eq13", "relL2")
    out = ["  ".join(f"{h:>12}" for h in head)]
    for r in rows:
        st = r["stage_us"]
        rel = r["rel_l2_vs_dense_per_step"]
        cells = (r["shape"][:12], r["variant"][:12], f"{r['keep']:.3f}", r["refresh"], f"{r['k_core']}+{r['k_anchor']}",
                 r["packed_len"], st["score"], st["select"], st["pack"], st["attn_packed"], st["scatter"], st["attn_dense"],
                 r["full_step_us"], r["sparse_step_us"] if r["sparse_step_us"] is not None else "-",
                 r["schedule_graph_us"] if r["schedule_graph_us"] is not None else "-", f"{r['tokens_per_s'] / 1e6:.2f}",
                 r["iou_consecutive_steps"] if r["iou_consecutive_steps"] is not None else "-",
                 r["overlap_eq13_consecutive_steps"], f"{max(rel):.3f}")
        out.append("  ".join(f"{str(c):>12}" for c in cells))
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--summarise", default="", help="print the JSON lines of an earlier run as a text table and exit")
    ap.add_argument("--shape", default="sweep", choices=["sweep"] + sorted(W.PAPER_SHAPES))
    ap.add_argument("--keeps", default=",".join(str(k) for k in W.SWEEP_KEEPS), help="keep ratios (shape 'sweep')")
    ap.add_argument("--budgets", default="", help="retained tokens per frame (paper shapes); default: the shape's own")
    ap.add_argument("--variants", default="combined", help="of " + ",".join(W.SELECT_VARIANTS))
    ap.add_argument("--refresh", default=",".join(str(r) for r in W.SWEEP_REFRESH),
                    help="refresh intervals; 'first' = only the first step is a full step")
    ap.add_argument("--steps", type=int, default=0, help="denoising steps (default: 10, or the paper shape's own)")
    args = ap.parse_args()
    if args.summarise:
        print(summarise(args.summarise))
        return
    variants = args.variants.split(",")
    if args.shape == "sweep":
        base = W.sweep_workload(1.0, 1)
        n_steps = args.steps or 10
        cases = [W.sweep_workload(float(k), 1) for k in args.keeps.split(",")]
    else:
        base = W.PAPER_SHAPES[args.shape]
        n_steps = args.steps or base.steps
        cases = [base] if not args.budgets else [W.variant_workload(base, "combined", int(k)) for k in args.budgets.split(",")]
    refreshes = [n_steps if r == "first" else int(r) for r in args.refresh.split(",")]
    base = base.with_(steps=n_steps)
    host = W.generate_steps(base, n_steps)                 # the inputs do not depend on budgets, variant or R
    dev_steps = [{n: swam.to_device(x[n], base.dtype) for n in "qkv"} for x in host]
    dense_ctx = swam.Swam.from_workload(base)
    dense_outs = [dense_ctx.sparse_attn(x["q"], x["k"], x["v"]) for x in dev_steps]   # memoised dense results
    for case in cases:
        for variant in variants:
            wl = W.variant_workload(case, variant).with_(steps=n_steps, name=f"{base.name}_k{case.k_keep}")
            for r in refreshes:
                print(json.dumps(run_config(wl.with_(refresh=r), r, n_steps, dev_steps, dense_outs, variant)), flush=True)


if __name__ == "__main__":
    main()
