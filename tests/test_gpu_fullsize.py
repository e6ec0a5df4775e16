"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (swam_step FULL then REUSE).

The oracle cannot finish every attention row at these sizes in seconds, so attention outputs are checked on sampled
rows that always include the first and last row of several 128-row tiles, the ragged tail tile and action rows;
scores, selections and maps are checked in full; packed tensors and omitted rows are checked exactly; and the
tcgen05 kernel is compared with the independent mma.sync kernel on every element.
"""
import numpy as np
import pytest
import torch

from oracle import reference as ora
from paper_2609_38984_b200 import workloads as W

pytestmark = pytest.mark.gpu


def sample_rows(rng, batch, n, n_random, extra=()):
    rows = {(0, 0), (batch - 1, n - 1)}
    for r in (127, 128, 255, 256, 383, (n // 128) * 128 - 1, (n // 128) * 128 % n, n - 2):
        if 0 <= r < n:
            rows.add((int(rng.integers(0, batch)), r))
    for r in extra:
        rows.add((int(rng.integers(0, batch)), int(r)))
    while len(rows) < n_random + 10:
        rows.add((int(rng.integers(0, batch)), int(rng.integers(0, n))))
    return np.array(sorted(rows), dtype=np.int32)


def check_bf16(got, want):
    err = np.abs(got - want)
    assert err.max() <= 2e-2, err.max()
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= 1e-2, rel


FULL_SIZE = [
    ("single_view", W.WORKLOADS["single_view"], 160),
    ("larger_imagination", W.WORKLOADS["larger_imagination"], 56),
    ("multi_view", W.WORKLOADS["multi_view"], 48),
    # the keep-ratio sweep at the larger-imagination shape (seed 4); 0.3 is the larger_imagination case above
    ("sweep_keep0.1", W.sweep_workload(0.1, 2), 40),
    ("sweep_keep0.2", W.sweep_workload(0.2, 2), 40),
    ("sweep_keep0.5", W.sweep_workload(0.5, 2), 40),
    ("sweep_keep1.0", W.sweep_workload(1.0, 2), 40),
]


@pytest.mark.parametrize("name,wl,n_rows", FULL_SIZE, ids=[c[0] for c in FULL_SIZE])
def test_full_size_cycle_matches_oracle(name, wl, n_rows):
    from paper_2609_38984_b200 import swam
    kc, ks = wl.budgets
    steps = W.generate_steps(wl, 2)
    x0, x1 = steps
    ctx = swam.Swam.from_workload(wl)
    out = ctx.empty_full().zero_()
    d0 = {n: swam.to_device(x0[n], wl.dtype) for n in "qkv"}
    d1 = {n: swam.to_device(x1[n], wl.dtype) for n in "qkv"}
    rng = np.random.default_rng(7)

    # ---- full step -------------------------------------------------------------------------------------
    ctx.step(d0["q"], d0["k"], d0["v"], swam.REFRESH_FULL, out)
    ctx.check()
    out_full = out.clone()
    sc_dev, lse_dev, _ = ctx.cached_scores()
    sel_dev, pm_dev, im_dev = (t.cpu().numpy().copy() for t in ctx.selection())
    lse64 = ora.action_lse(x0["q"], x0["k"], wl.n_action)
    assert np.abs(lse_dev.cpu().numpy() - lse64).max() <= 2e-3          # normalisers from the bf16 dense pass
    s64 = ora.score(x0["q"], x0["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse64)
    got_s = sc_dev.cpu().numpy()
    # scores inherit the dense kernel's fp32 normaliser (error e-6 absolute in the exponent)
    rel = np.abs(got_s - s64) / np.maximum(s64, 1e-30)
    assert rel.max() <= 1e-5, rel.max()
    iso = ora.select(got_s, kc, ks)
    ipm, iim = ora.maps(iso["sel_idx"], wl.n_obs, wl.n_spatial, wl.n_action)
    assert np.array_equal(sel_dev, iso["sel_idx"]) and np.array_equal(pm_dev, ipm) and np.array_equal(im_dev, iim)
    e2e = ora.select(s64.astype(np.float32), kc, ks)
    assert np.array_equal(sel_dev, e2e["sel_idx"]), ("cut margins", e2e["margins"], "score rel err", rel.max())
    action_rows = range(wl.seq_len - wl.n_action, wl.seq_len, max(1, wl.n_action // 6))
    rows = sample_rows(rng, wl.batch, wl.seq_len, n_rows, extra=action_rows)
    want, _ = ora.attention_rows(x0["q"], x0["k"], x0["v"], rows)
    got = out_full[rows[:, 0], rows[:, 1]].float().cpu().numpy().astype(np.float64)
    check_bf16(got, want)

    # ---- sparse step -----------------------------------------------------------------------------------
    ctx.step(d1["q"], d1["k"], d1["v"], swam.REUSE, out)
    ctx.check()
    # packed tensors are exact gathers
    pm_t = torch.from_numpy(pm_dev).cuda()
    qp, kp, vp = ctx.pack(d1["q"], d1["k"], d1["v"], pm_t)
    for src, gotp in ((x1["q"], qp), (x1["k"], kp), (x1["v"], vp)):
        assert np.array_equal(gotp.float().cpu().numpy(), ora.pack(src, pm_dev))
    # omitted rows keep the full step's values bit for bit; retained rows changed
    omitted = torch.from_numpy(im_dev < 0).cuda()
    assert int(omitted.sum()) == wl.batch * (wl.seq_len - wl.packed_len)
    if wl.packed_len < wl.seq_len:
        assert torch.equal(out[omitted], out_full[omitted])
    else:
        assert np.array_equal(pm_dev[0], np.arange(wl.seq_len))     # keep ratio 1.0: identity map
    rows_p = sample_rows(rng, wl.batch, wl.packed_len, n_rows, extra=range(wl.packed_len - wl.n_action, wl.packed_len, 8))
    qpo, kpo, vpo = ora.pack(x1["q"], pm_dev), ora.pack(x1["k"], pm_dev), ora.pack(x1["v"], pm_dev)
    want_p, _ = ora.attention_rows(qpo, kpo, vpo, rows_p)
    orig = pm_dev[rows_p[:, 0], rows_p[:, 1]]
    got_p = out[rows_p[:, 0], orig].float().cpu().numpy().astype(np.float64)
    check_bf16(got_p, want_p)

    # ---- the fused sparse step (scatter inside the attention kernel) equals the staged one bit for bit -------
    staged = swam.Swam.from_workload(wl)
    staged.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_STAGED)
    out_s = out_full.clone()
    staged.step(d0["q"], d0["k"], d0["v"], swam.REFRESH_FULL, out_s)
    staged.step(d1["q"], d1["k"], d1["v"], swam.REUSE, out_s)
    staged.check()
    assert torch.equal(out_s, out)
    del staged, out_s
    # ... and so does the variant in which the kernel gathers the key and value rows itself
    gkv = swam.Swam.from_workload(wl)
    gkv.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_FUSED_KV)
    out_g = out_full.clone()
    gkv.step(d0["q"], d0["k"], d0["v"], swam.REFRESH_FULL, out_g)
    gkv.step(d1["q"], d1["k"], d1["v"], swam.REUSE, out_g)
    gkv.check()
    assert torch.equal(out_g, out)
    del gkv, out_g

    # ---- every element: tcgen05 kernel vs the independent mma.sync kernel ----------------------------------
    other = swam.Swam.from_workload(wl)
    other.set_option(swam.OPT_ATTN_VARIANT, swam.ATTN_WARP_MMA)
    ref_p, ref_lse = other.sparse_attn(qp, kp, vp, want_lse=True)
    tc_p, tc_lse = ctx.sparse_attn(qp, kp, vp, want_lse=True)
    ctx.check()
    diff = (ref_p.float() - tc_p.float()).abs()
    assert float(diff.max()) <= 2e-2
    assert float(diff.norm() / ref_p.float().norm()) <= 5e-3
    assert float((ref_lse - tc_lse).abs().max()) <= 1e-3
    ref_d = other.sparse_attn(d0["q"], d0["k"], d0["v"])
    diff = (ref_d.float() - out_full.float()).abs()
    assert float(diff.max()) <= 2e-2
    assert float(diff.norm() / ref_d.float().norm()) <= 5e-3


def test_attention_is_deterministic_at_full_size():
    from paper_2609_38984_b200 import swam
    wl = W.WORKLOADS["larger_imagination"]
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    q, k, v = (swam.to_device(x[n], wl.dtype)[:, :wl.packed_len].contiguous() for n in "qkv")
    first = ctx.sparse_attn(q, k, v)
    for _ in range(5):
        assert torch.equal(first, ctx.sparse_attn(q, k, v))
    ctx.check()


@pytest.mark.parametrize("name", ["single_view", "larger_imagination", "multi_view"])
def test_full_size_light_refresh_matches_oracle(name):
    """SWAM_REFRESH_LIGHT at the benchmark sizes: the one-pass scorer's normalisers and scores (every element) and
    the selection and maps built from them against the oracle, then the packed attention's retained rows on a seeded
    sample and the omitted rows bit for bit."""
    from paper_2609_38984_b200 import swam
    wl = W.WORKLOADS[name]
    kc, ks = wl.budgets
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    out = ctx.empty_full()
    out.copy_(torch.randn(out.shape, device="cuda", generator=torch.Generator(device="cuda").manual_seed(3)).to(out.dtype))
    before = out.clone()
    q, k, v = (swam.to_device(x[n], wl.dtype) for n in "qkv")
    ctx.step(q, k, v, swam.REFRESH_LIGHT, out)
    ctx.check()
    sc_dev, lse_dev, _ = ctx.cached_scores()
    sel_dev, pm_dev, im_dev = (t.cpu().numpy().copy() for t in ctx.selection())
    lse64 = ora.action_lse(x["q"], x["k"], wl.n_action)
    assert np.abs(lse_dev.cpu().numpy() - lse64).max() <= 1e-4          # fp32 running sums over bf16 products
    s64 = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse64)
    got_s = sc_dev.cpu().numpy()
    rel = np.abs(got_s - s64) / np.maximum(s64, 1e-30)
    assert np.isfinite(got_s).all() and rel.max() <= 1e-5, rel.max()
    iso = ora.select(got_s, kc, ks)
    ipm, iim = ora.maps(iso["sel_idx"], wl.n_obs, wl.n_spatial, wl.n_action)
    assert np.array_equal(sel_dev, iso["sel_idx"]) and np.array_equal(pm_dev, ipm) and np.array_equal(im_dev, iim)
    e2e = ora.select(s64.astype(np.float32), kc, ks)
    assert np.array_equal(sel_dev, e2e["sel_idx"]), ("cut margins", e2e["margins"], "score rel err", rel.max())
    omitted = torch.from_numpy(im_dev < 0).cuda()
    assert torch.equal(out[omitted], before[omitted])
    qp, kp, vp = (ora.pack(x[n], pm_dev) for n in "qkv")
    rng = np.random.default_rng(11)
    rows = sample_rows(rng, wl.batch, wl.packed_len, 40, extra=range(wl.packed_len - wl.n_action, wl.packed_len, 8))
    want, _ = ora.attention_rows(qp, kp, vp, rows)
    orig = pm_dev[rows[:, 0], rows[:, 1]]
    got = out[rows[:, 0], orig].float().cpu().numpy().astype(np.float64)
    check_bf16(got, want)
