"""Parity of the CUDA path (through the C-ABI) against the CPU oracle, stage by stage and end to end.

Bars: selected indices, pack maps and inverse maps bit-exact; packed/scattered tensors bit-exact; scores within
1e-4 max-abs and 1e-5 relative; attention outputs within 1e-4 max-abs (fp32) or 2e-2 max-abs with relative
L2 <= 1e-2 (bf16).
"""
import numpy as np
import pytest
import torch

from oracle import reference as ora
from paper_2609_38984_b200 import workloads as W

pytestmark = pytest.mark.gpu

SCORE_REL = 1e-5


def _swam():
    from paper_2609_38984_b200 import swam
    return swam


def small(name="single_view", **kw):
    base = dict(n_obs=70, grid_h=10, grid_w=9, n_heads=3, steps=3)
    base.update(kw)
    return W.WORKLOADS[name].with_(**base)


def dev(x, wl):
    return _swam().to_device(x, wl.dtype)


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def check_float(got, want, dtype):
    err = np.abs(got - want)
    if dtype == W.F32:
        assert err.max() <= 1e-4, err.max()
    else:
        assert err.max() <= 2e-2, err.max()
        rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
        assert rel <= 1e-2, rel


# ------------------------------------------------------------------ select
SELECT_SHAPES = [
    # (B, F, N_s, K_c, K_s, n_obs, H)
    (1, 2, 64, 14, 18, 16, 8),            # tiny
    (3, 4, 90, 10, 13, 7, 32),            # ragged N_s
    (2, 8, 360, 80, 104, 33, 32),         # the paper's 360-token frames with 80 + 104
    (1, 2, 98, 19, 12, 5, 32),            # the paper's 98-token frames with 19 + 12
    (1, 8, 1024, 133, 174, 1024, 64),     # larger-imagination shape
    (8, 4, 1728, 188, 244, 1728, 32),     # multi-view shape
    (1, 3, 50, 7, 0, 0, 3),               # no anchors, F not a power of two, no observed tokens
    (1, 3, 50, 0, 9, 4, 3),               # no core tokens
    (2, 5, 40, 15, 25, 4, 5),             # keep everything
    (1, 1, 33, 4, 5, 2, 4),               # a single frame
]


@pytest.mark.parametrize("shape", SELECT_SHAPES)
@pytest.mark.parametrize("ties", [False, True])
def test_select_bit_exact(shape, ties):
    swam = _swam()
    B, F, N, kc, ks, n_obs, H = shape
    s = W.random_scores(17 + N, B, F, N, ties=ties)
    ctx = swam.Swam(B, n_obs, F, N, H, 2, 32, kc, ks, dtype=swam.F32, query_weights=[1.0 / (H // F)] * (H // F))
    sel, pack, inv = ctx.select(torch.from_numpy(s).cuda())
    ctx.check()
    want = ora.select(s, kc, ks)
    wp, wi = ora.maps(want["sel_idx"], n_obs, N, H)
    assert np.array_equal(sel.cpu().numpy(), want["sel_idx"])
    assert np.array_equal(pack.cpu().numpy(), wp)
    assert np.array_equal(inv.cpu().numpy(), wi)


def test_select_all_equal_and_zero_scores():
    swam = _swam()
    for val in (0.0, 0.25):
        s = np.full((2, 4, 70), val, np.float32)
        ctx = swam.Swam(2, 3, 4, 70, 8, 2, 32, 9, 11, dtype=swam.F32, query_weights=[0.5, 0.5])
        sel, pack, inv = ctx.select(torch.from_numpy(s).cuda())
        ctx.check()
        want = ora.select(s, 9, 11)
        assert np.array_equal(sel.cpu().numpy(), want["sel_idx"])
        assert sel.cpu().numpy()[0, 0].tolist() == list(range(20))


def test_select_is_deterministic():
    swam = _swam()
    s = torch.from_numpy(W.random_scores(3, 4, 8, 512, ties=True)).cuda()
    ctx = swam.Swam(4, 10, 8, 512, 64, 2, 32, 60, 80, dtype=swam.F32)
    first = [t.clone() for t in ctx.select(s)]
    for _ in range(20):
        again = ctx.select(s)
        for a, b in zip(first, again):
            assert torch.equal(a, b)


# ------------------------------------------------------------------ score
@pytest.mark.parametrize("wl", [
    W.WORKLOADS["tiny"],
    small(),                                              # bf16, D = 64, g = 8, ragged frame size
    small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=5),   # bf16, D = 128
    small(n_frames=2, n_action=32, head_dim=32),          # g = 16 (two query tiles), D = 32
    small(n_frames=8, n_action=32),                       # g = 4 (padded query tile)
    small(n_frames=10, n_action=40),                      # H = 40: more than two 16-row query blocks, fewer than four
    small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=5, n_frames=3, n_action=48),   # H = 48, g = 16
], ids=["tiny_f32", "d64", "d128", "g16_d32", "g4", "h40", "h48_g16_d128"])
@pytest.mark.parametrize("given_lse", [True, False])
def test_score_matches_oracle(wl, given_lse):
    swam = _swam()
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    q, k = dev(x["q"], wl), dev(x["k"], wl)
    lse64 = ora.action_lse(x["q"], x["k"], wl.n_action)
    lse_t = torch.from_numpy(lse64.astype(np.float32)).cuda() if given_lse else None
    s, qual = ctx.score(q, k, lse_t, quality=True)
    ctx.check()
    want = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse64)
    got = s.cpu().numpy().astype(np.float64)
    assert np.abs(got - want).max() <= 1e-4
    rel = np.abs(got - want) / np.maximum(want, 1e-30)
    assert rel.max() <= SCORE_REL, rel.max()
    wq = ora.quality(want.astype(np.float32))
    assert np.allclose(qual.cpu().numpy(), wq, rtol=1e-4, atol=1e-6)
    if not given_lse:
        _, lse_dev, _ = ctx.cached_scores()
        assert np.abs(lse_dev.cpu().numpy() - lse64).max() <= 1e-4


@pytest.mark.parametrize("n_frames,n_action", [(10, 40), (12, 48), (3, 48)], ids=["h40", "h48_g4", "h48_g16"])
def test_normalisers_computed_on_the_device_cover_every_action_row(n_frames, n_action):
    """Action counts between 33 and 63 need all four 16-row query blocks of the normaliser kernel: the scores of
    swam_score (no normalisers given), of swam_score_noalloc and of a light refresh step are checked on them."""
    swam = _swam()
    wl = small(n_frames=n_frames, n_action=n_action)
    x = W.generate_steps(wl, 1)[0]
    q, k, v = (dev(x[n], wl) for n in "qkv")
    lse64 = ora.action_lse(x["q"], x["k"], wl.n_action)
    want = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse64)
    ctx = swam.Swam.from_workload(wl)
    got = {"score": ctx.score(q, k).cpu().numpy().astype(np.float64)}
    _, lse_dev, _ = ctx.cached_scores()
    assert np.abs(lse_dev.cpu().numpy() - lse64).max() <= 1e-4
    na = torch.full((wl.batch, wl.n_frames, wl.n_spatial), float("nan"), device="cuda")
    swam.Swam.from_workload(wl, bind=False).score_noalloc(q, k, na)
    got["noalloc"] = na.cpu().numpy().astype(np.float64)
    out = ctx.empty_full().zero_()
    ctx.step(q, k, v, swam.REFRESH_LIGHT, out)
    ctx.check()
    got["light"] = ctx.cached_scores()[0].cpu().numpy().astype(np.float64)
    for name, g in got.items():
        rel = np.abs(g - want) / np.maximum(want, 1e-30)
        assert np.isfinite(g).all() and rel.max() <= SCORE_REL, (name, rel.max())


ONE_PASS_CASES = [
    # the one-pass scorer's branches: copies of the query chunk in the tile (4, 2, 1), more than one chunk, side-output
    # rows that start off a 16-byte boundary, frames shorter and longer than a key tile, several key ranges per head
    ("single_view", dict(n_obs=70, grid_h=10, grid_w=9, n_heads=3), None, None),                      # H = 32: 4 copies
    ("single_view", dict(n_obs=41, grid_h=7, grid_w=9, n_heads=2, batch=2), None, None),              # odd offsets: scalar stores
    ("single_view", dict(n_obs=600, grid_h=16, grid_w=17, n_heads=2, n_frames=8, n_action=64), None, None),     # H = 64: 2 copies
    ("larger_imagination", dict(n_obs=300, grid_h=12, grid_w=12, n_heads=2, n_frames=6, n_action=96), None, None),   # H = 96: 1 copy
    ("larger_imagination", dict(n_obs=64, grid_h=6, grid_w=6, n_heads=2, n_frames=5, n_action=160), None, None),     # two chunks
    ("larger_imagination", dict(n_obs=40, grid_h=5, grid_w=5, n_heads=3, n_frames=8, n_action=8), [1.0], None),     # g = 1
    ("single_view", dict(n_obs=128, grid_h=8, grid_w=8, n_heads=4, n_frames=4, n_action=8), [0.25, 0.75], None),    # g = 2
    ("single_view", dict(n_obs=2000, grid_h=24, grid_w=24, n_heads=4, n_kv_heads=2), None, (0, 1, 1)),               # GQA, action rows do not see action keys
]


@pytest.mark.parametrize("name,kw,alpha,sees", ONE_PASS_CASES,
                         ids=["h32", "odd_offsets", "h64", "h96", "h160", "g1", "g2", "gqa_no_action_keys"])
def test_one_pass_scorer_matches_oracle(name, kw, alpha, sees):
    """swam_score without given normalisers on the tensor-core path: one stream over K yields the normalisers and the
    future keys' products, a second kernel the scores (Eq. 12); both are compared with the oracle on every element."""
    swam = _swam()
    wl = W.WORKLOADS[name].with_(**kw)
    x = W.generate_steps(wl, 1)[0]
    kc, ks = wl.budgets
    ctx = swam.Swam(wl.batch, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, wl.n_heads, wl.head_dim, kc, ks,
                    dtype=wl.dtype, n_kv_heads=wl.kv_heads, query_weights=alpha)
    n_visible = None
    if sees is not None:
        ctx.set_visibility(*sees)
        n_visible = [wl.n_obs, wl.n_obs + wl.n_frames * wl.n_spatial, wl.seq_len][sees[2]]
    q, k = dev(x["q"], wl), dev(x["k"], wl)
    k64 = ora.expand_kv(x["k"], wl.n_heads)
    lse64 = ora.action_lse(x["q"], k64, wl.n_action, n_visible=n_visible)
    want = ora.score(x["q"], k64, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse64,
                     alpha=None if alpha is None else np.array(alpha))
    first = None
    for rep in range(2):      # the second call finds the arrival tickets as the first one left them
        got_t = ctx.score(q, k)
        got = got_t.cpu().numpy().astype(np.float64)
        ctx.check()
        if first is None:
            first = got_t.clone()
        else:
            assert torch.equal(first, got_t)      # same bits whatever order the key ranges finish in
        _, lse_dev, _ = ctx.cached_scores()
        assert np.abs(lse_dev.cpu().numpy() - lse64).max() <= 1e-4, rep
        rel = np.abs(got - want) / np.maximum(want, 1e-30)
        assert np.isfinite(got).all() and rel.max() <= SCORE_REL, (rep, rel.max())


def test_score_custom_weights():
    swam = _swam()
    wl = small(n_frames=4, n_action=12)                   # g = 3: only valid with explicit weights
    x = W.generate_steps(wl, 1)[0]
    alpha = [0.2, 0.5, 0.3]
    kc, ks = wl.budgets
    with pytest.raises(swam.SwamError):
        swam.Swam.from_workload(wl)
    ctx = swam.Swam(wl.batch, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, wl.n_heads, wl.head_dim, kc, ks,
                    dtype=wl.dtype, query_weights=alpha)
    s = ctx.score(dev(x["q"], wl), dev(x["k"], wl))
    want = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, alpha=np.array(alpha))
    rel = np.abs(s.cpu().numpy() - want) / want
    assert rel.max() <= SCORE_REL


# ------------------------------------------------------------------ pack / scatter
@pytest.mark.parametrize("wl", [W.WORKLOADS["tiny"], small(batch=2)], ids=["f32", "bf16"])
def test_pack_and_scatter_exact(wl):
    swam = _swam()
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    kc, ks = wl.budgets
    sc = W.random_scores(5, wl.batch, wl.n_frames, wl.n_spatial)
    sel = ora.select(sc, kc, ks)["sel_idx"]
    pm, im = ora.maps(sel, wl.n_obs, wl.n_spatial, wl.n_action)
    pm_t, im_t = torch.from_numpy(pm).cuda(), torch.from_numpy(im).cuda()
    q, k, v = (dev(x[n], wl) for n in "qkv")
    qp, kp, vp = ctx.pack(q, k, v, pm_t)
    for src, got in ((x["q"], qp), (x["k"], kp), (x["v"], vp)):
        assert np.array_equal(got.float().cpu().numpy(), ora.pack(src, pm))
    only_k = ctx.pack(None, k, None, pm_t)
    assert only_k[0] is None and torch.equal(only_k[1], kp)
    # in place: retained rows replaced, omitted rows untouched
    cached = dev(x["v"], wl)
    before = cached.clone()
    ctx.scatter(qp, pm_t, im_t, cached)
    want = ora.scatter(ora.pack(x["q"], pm), pm, x["v"])
    assert np.array_equal(cached.float().cpu().numpy(), want)
    # blend into a fresh buffer
    out = torch.zeros_like(before)
    ctx.scatter(qp, pm_t, im_t, before, out)
    assert np.array_equal(out.float().cpu().numpy(), want)
    ctx.check()


def test_corrupt_map_is_reported_not_followed():
    swam = _swam()
    wl = small()
    ctx = swam.Swam.from_workload(wl)
    x = W.generate_steps(wl, 1)[0]
    pm = torch.arange(wl.packed_len, dtype=torch.int32).repeat(wl.batch, 1).cuda()
    pm[0, 5] = wl.seq_len + 3
    pm[0, 6] = -2
    q = dev(x["q"], wl)
    qp = ctx.pack(q, None, None, pm)[0]
    with pytest.raises(swam.SwamError) as e:
        ctx.check()
    assert e.value.code == swam.ERR_DEVICE_CHECK
    ctx.check()     # the status word was cleared
    assert torch.equal(qp[0, 7], q[0, 7])


# ------------------------------------------------------------------ attention
ATTN_CASES = [
    ("tiny", dict()),
    ("tiny", dict(n_obs=3, head_dim=64)),
    ("single_view", dict(n_obs=70, grid_h=10, grid_w=9, n_heads=3)),                 # D = 64, L = 462
    ("single_view", dict(n_obs=1, grid_h=4, grid_w=4, n_heads=2, n_action=16, head_dim=32)),
    ("larger_imagination", dict(n_obs=40, grid_h=7, grid_w=9, n_heads=2, batch=2)),    # D = 128, L = 608
    ("larger_imagination", dict(n_obs=0, grid_h=2, grid_w=2, n_heads=1, n_action=32)),  # L = 64: one tile
    ("larger_imagination", dict(n_obs=1, grid_h=2, grid_w=2, n_heads=1, n_action=32)),  # L = 65
]


@pytest.mark.parametrize("name,kw", ATTN_CASES)
def test_attention_matches_oracle(name, kw):
    swam = _swam()
    wl = W.WORKLOADS[name].with_(**kw)
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    q, k, v = (dev(x[n], wl) for n in "qkv")
    out, lse = ctx.sparse_attn(q, k, v, want_lse=True)
    ctx.check()
    want, wlse = ora.attention(x["q"], x["k"], x["v"])
    check_float(f64(out), want, wl.dtype)
    assert np.abs(lse.cpu().numpy() - wlse).max() <= (1e-4 if wl.dtype == W.F32 else 2e-3)


@pytest.mark.parametrize("head_dim", [32, 64, 128])
@pytest.mark.parametrize("pattern", ["ramp", "late_spike"])
def test_attention_with_a_growing_row_maximum(head_dim, pattern):
    """Logits that keep outgrowing the maximum of the first key tile: every later tile (ramp) or one late tile
    (late_spike) forces the running reference of the online softmax to be raised and the output rescaled."""
    swam = _swam()
    n = 1100                                   # nine key tiles, ragged tail
    wl = W.WORKLOADS["single_view"].with_(n_obs=n - 64 - 32, grid_h=8, grid_w=8, n_frames=1, n_action=32, n_heads=2,
                                          head_dim=head_dim, keep=1.0)
    assert wl.seq_len == n
    rng = np.random.default_rng(5)
    shape = (1, n, 2, head_dim)
    u = rng.standard_normal(head_dim)
    u /= np.linalg.norm(u)
    # q = noise + sqrt(D) u and k = noise + gain u give a logit of about `gain` (natural-log units)
    q = 0.3 * rng.standard_normal(shape) + u * np.sqrt(head_dim)
    pos = np.arange(n)[None, :, None, None]
    if pattern == "ramp":
        gain = 12.0 * (pos // 128)             # far beyond the 2^8 slack of the running reference, at every tile
    else:
        gain = np.where((pos >= 700) & (pos < 720), 40.0, 0.0)
    k = 0.3 * rng.standard_normal(shape) + u * gain
    v = rng.standard_normal(shape)
    q, k, v = (t.astype(np.float32) for t in (q, k, v))
    ctx = swam.Swam.from_workload(wl)
    qd, kd, vd = (dev(t, wl) for t in (q, k, v))
    qh, kh, vh = (f64(t) for t in (qd, kd, vd))          # the bf16-rounded values the kernel sees
    out, lse = ctx.sparse_attn(qd, kd, vd, want_lse=True)
    ctx.check()
    want, wlse = ora.attention(qh, kh, vh)
    check_float(f64(out), want, wl.dtype)
    assert np.abs(lse.cpu().numpy() - wlse).max() <= 5e-3
    # several passes: the result does not depend on timing between the roles of the kernel
    for _ in range(5):
        again = ctx.sparse_attn(qd, kd, vd)
        assert torch.equal(again, out)


@pytest.mark.parametrize("head_dim,n_heads,n", [
    (64, 50, 768),       # 150 work items on 148 SMs: two left over, cut over the keys
    (64, 37, 2048),      # 296 items: exactly two per CTA
    (128, 38, 2148),     # 342 items: two per CTA and 46 left over (split), ragged last tile
    (128, 5, 4000),      # 80 items: fewer than SMs
])
def test_attention_work_distribution_over_persistent_ctas(head_dim, n_heads, n):
    """Item counts below, at and just above multiples of the SM count: the CTAs walk through several items each and
    the leftover items are cut over the keys and merged; every element is compared with the mma.sync kernel, sampled
    rows with the oracle."""
    swam = _swam()
    wl = W.WORKLOADS["single_view"].with_(n_obs=n - 64 - 32, grid_h=8, grid_w=8, n_frames=1, n_action=32,
                                          n_heads=n_heads, head_dim=head_dim, keep=1.0, seed=21)
    assert wl.seq_len == n
    x = W.generate_steps(wl, 1)[0]
    q, k, v = (dev(x[m], wl) for m in "qkv")
    tc = swam.Swam.from_workload(wl)
    ref = swam.Swam.from_workload(wl)
    ref.set_option(swam.OPT_ATTN_VARIANT, swam.ATTN_WARP_MMA)
    out, lse = tc.sparse_attn(q, k, v, want_lse=True)
    out_r, lse_r = ref.sparse_attn(q, k, v, want_lse=True)
    tc.check()
    diff = (out.float() - out_r.float()).abs()
    assert float(diff.max()) <= 2e-2 and float(diff.norm() / out_r.float().norm()) <= 5e-3
    assert float((lse - lse_r).abs().max()) <= 1e-3
    rng = np.random.default_rng(3)
    rows = np.stack([np.zeros(24, np.int32), rng.integers(0, n, 24).astype(np.int32)], axis=1)
    rows[0, 1], rows[1, 1], rows[2, 1] = 0, n - 1, min((n // 256) * 256, n - 1)
    assert rows[:, 1].min() >= 0 and rows[:, 1].max() < n
    want, _ = ora.attention_rows(x["q"], x["k"], x["v"], rows)
    check_float(f64(out[rows[:, 0], rows[:, 1]]), want, wl.dtype)
    assert torch.equal(out, tc.sparse_attn(q, k, v))          # and the same bits again


@pytest.mark.parametrize("name,lengths", [
    ("single_view", (1, 2, 63, 64, 65, 127, 129, 200)),
    # head dim 128: one to five key tiles, i.e. every start-up sequence of the ring that K and V tiles share there
    ("larger_imagination", (1, 127, 128, 129, 256, 257, 384, 385, 513, 600)),
], ids=["d64", "d128"])
def test_attention_short_sequences(name, lengths):
    """seq_len below the full length, down to one token."""
    swam = _swam()
    wl = small(name, n_obs=160, grid_h=10, grid_w=9, n_heads=3) if name != "single_view" else small()
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    assert max(lengths) <= wl.seq_len
    for n in lengths:
        q, k, v = (dev(np.ascontiguousarray(x[m][:, :n]), wl) for m in "qkv")
        out = ctx.sparse_attn(q, k, v)
        want, _ = ora.attention(x["q"][:, :n], x["k"][:, :n], x["v"][:, :n])
        check_float(f64(out), want, wl.dtype)


# ------------------------------------------------------------------ whole steps
def run_schedule(ctx, wl, steps, refresh):
    swam = _swam()
    out = ctx.empty_full().zero_()
    log = []
    for t, x in enumerate(steps):
        mode = swam.REFRESH_FULL if t % refresh == 0 else swam.REUSE
        ctx.step(dev(x["q"], wl), dev(x["k"], wl), dev(x["v"], wl), mode, out)
        ctx.check()
        sel, pm, im = ctx.selection()
        sc, _, _ = ctx.cached_scores()
        log.append(dict(out=f64(out), sel=sel.cpu().numpy().copy(), pm=pm.cpu().numpy().copy(),
                        im=im.cpu().numpy().copy(), scores=sc.cpu().numpy().copy()))
    return log


def compare_schedule(wl, steps, refresh, log):
    """Oracle run that follows the paper's step loop; index equality is required unless a TopK cut is closer
    than the score error can resolve, in which case the case is reported by the assertion message."""
    kc, ks = wl.budgets
    want = ora.run_steps(steps, refresh, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, kc, ks)
    for t, (g, w) in enumerate(zip(log, want)):
        rel = np.abs(g["scores"] - w["scores"].astype(np.float64)) / np.maximum(w["scores"], 1e-30)
        assert rel.max() <= SCORE_REL, (t, rel.max())
        # stage-isolated exactness: the GPU selection equals the oracle's selection of the GPU's own scores
        iso = ora.select(g["scores"], kc, ks)
        ipm, iim = ora.maps(iso["sel_idx"], wl.n_obs, wl.n_spatial, wl.n_action)
        assert np.array_equal(g["sel"], iso["sel_idx"]) and np.array_equal(g["pm"], ipm) and np.array_equal(g["im"], iim)
        # end to end
        assert np.array_equal(g["sel"], w["sel_idx"]), (t, "cut margins", w["margins"], "score rel err", rel.max())
        assert np.array_equal(g["pm"], w["pack_map"]) and np.array_equal(g["im"], w["inv_map"])
        check_float(g["out"], w["out"], wl.dtype)


def test_tiny_schedule_matches_oracle():
    swam = _swam()
    wl = W.WORKLOADS["tiny"]
    steps = W.generate_steps(wl)
    ctx = swam.Swam.from_workload(wl)
    compare_schedule(wl, steps, wl.refresh, run_schedule(ctx, wl, steps, wl.refresh))


@pytest.mark.parametrize("wl", [
    small(batch=2),
    small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=2, steps=3),
    small("multi_view", batch=2, n_obs=33, grid_h=5, grid_w=4, n_heads=2, steps=4),
], ids=["d64", "d128", "multiview"])
def test_bf16_schedule_matches_oracle(wl):
    swam = _swam()
    steps = W.generate_steps(wl)
    ctx = swam.Swam.from_workload(wl)
    compare_schedule(wl, steps, wl.refresh, run_schedule(ctx, wl, steps, wl.refresh))


def test_refresh_every_step_and_keep_all():
    swam = _swam()
    wl = small(steps=2)
    steps = W.generate_steps(wl)
    ctx = swam.Swam.from_workload(wl)
    log = run_schedule(ctx, wl, steps, 1)
    compare_schedule(wl, steps, 1, log)
    # keep ratio 1.0: the sparse step runs over the identity map and reproduces dense attention
    wl1 = wl.with_(keep=1.0)
    ctx1 = swam.Swam.from_workload(wl1)
    log1 = run_schedule(ctx1, wl1, steps, 2)
    assert np.array_equal(log1[1]["pm"][0], np.arange(wl1.seq_len))
    dense, _ = ora.attention(steps[1]["q"], steps[1]["k"], steps[1]["v"])
    check_float(log1[1]["out"], dense, wl1.dtype)


def test_light_refresh_step():
    """score (normalisers computed on the device) -> select -> pack -> attention -> scatter in one call."""
    swam = _swam()
    wl = small()
    steps = W.generate_steps(wl, 2)
    ctx = swam.Swam.from_workload(wl)
    kc, ks = wl.budgets
    out = ctx.empty_full()
    x0, x1 = steps
    ctx.step(dev(x0["q"], wl), dev(x0["k"], wl), dev(x0["v"], wl), swam.REFRESH_FULL, out)
    ctx.step(dev(x1["q"], wl), dev(x1["k"], wl), dev(x1["v"], wl), swam.REFRESH_LIGHT, out)
    ctx.check()
    st = ora.full_step(ora.StepState(), x0["q"], x0["k"], x0["v"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, kc, ks)
    s1 = ora.score(x1["q"], x1["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action).astype(np.float32)
    st.scores = s1
    st.sel = ora.select(s1, kc, ks)
    st.pack_map, st.inv_map = ora.maps(st.sel["sel_idx"], wl.n_obs, wl.n_spatial, wl.n_action)
    ora.sparse_step(st, x1["q"], x1["k"], x1["v"])
    sel, pm, _ = ctx.selection()
    assert np.array_equal(sel.cpu().numpy(), st.sel["sel_idx"]), st.sel["margins"]
    check_float(f64(out), st.out, wl.dtype)


@pytest.mark.parametrize("wl", [
    small(batch=2),
    small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=2),
    small("larger_imagination", n_obs=300, grid_h=12, grid_w=11, n_heads=2, keep=0.5),   # whole tiles of observed rows
    small(n_obs=260, batch=2, n_heads=4, n_kv_heads=2),                                    # the same at head dim 64, grouped heads
    small(keep=1.0),
    small(keep=0.0),
], ids=["d64", "d128", "d128_long_obs", "d64_long_obs_gqa", "keep_all", "keep_none"])
@pytest.mark.parametrize("mode", ["reuse", "light"])
def test_fused_sparse_step_equals_staged_bit_for_bit(wl, mode):
    """Packed attention with the scatter and the query gather fused in, the same with the key and value rows gathered
    by the kernel as well, and pack -> attention -> scatter give the same bits."""
    swam = _swam()
    x0, x1 = W.generate_steps(wl, 2)
    outs = []
    for path in (swam.SPARSE_FUSED, swam.SPARSE_STAGED, swam.SPARSE_FUSED_KV):
        ctx = swam.Swam.from_workload(wl)
        ctx.set_option(swam.OPT_SPARSE_PATH, path)
        out = ctx.empty_full().zero_()
        n0 = ctx.launch_count()
        ctx.step(dev(x0["q"], wl), dev(x0["k"], wl), dev(x0["v"], wl), swam.REFRESH_FULL, out)
        n1 = ctx.launch_count()
        ctx.step(dev(x1["q"], wl), dev(x1["k"], wl), dev(x1["v"], wl),
                 swam.REUSE if mode == "reuse" else swam.REFRESH_LIGHT, out)
        ctx.check()
        outs.append((out.clone(), ctx.launch_count() - n1))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[2][0], outs[1][0])
    assert outs[2][1] < outs[0][1] < outs[1][1]          # each degree of fusion launches fewer kernels


# ------------------------------------------------------------------ ablations and shapes of the paper's evaluation
def _paper_shape(name, **kw):
    base = dict(n_heads=2)
    base.update(kw)
    return W.PAPER_SHAPES[name].with_(**base)


@pytest.mark.parametrize("variant", W.SELECT_VARIANTS)
@pytest.mark.parametrize("k_keep", W.PAPER_PRUNING_BUDGETS)
def test_selection_variants_at_the_paper_budgets(variant, k_keep):
    """Sec. 5.4's strategies (combined, core only, stable anchors only, random) at 256 / 184 / 112 of 360 tokens."""
    swam = _swam()
    wl = W.variant_workload(_paper_shape("cosmos3_nano"), variant, k_keep)
    kc, ks = wl.budgets
    ctx = swam.Swam.from_workload(wl)
    if variant == "random":
        scores = W.random_scores(77 + k_keep, wl.batch, wl.n_frames, wl.n_spatial)
    else:
        x = W.generate_steps(wl, 1)[0]
        scores = ctx.score(dev(x["q"], wl), dev(x["k"], wl)).cpu().numpy()
    sel, pm, im = ctx.select(torch.from_numpy(scores).cuda())
    ctx.check()
    want = ora.select(scores, kc, ks)
    wpm, wim = ora.maps(want["sel_idx"], wl.n_obs, wl.n_spatial, wl.n_action)
    assert np.array_equal(sel.cpu().numpy(), want["sel_idx"])
    assert np.array_equal(pm.cpu().numpy(), wpm) and np.array_equal(im.cpu().numpy(), wim)
    assert sel.shape[-1] == k_keep
    if variant == "stable_only":
        # shared anchors only: every frame keeps the same spatial indices
        s = sel.cpu().numpy()
        assert (s == s[:, :1]).all()


@pytest.mark.parametrize("name", ["cosmos3_nano", "cosmos3_edge", "fastwam_joint"])
def test_paper_shapes_with_only_the_first_step_full(name):
    """The default schedule of Sec. 4.2: one full step, every later step of the action chunk sparse."""
    swam = _swam()
    wl = _paper_shape(name)
    steps = W.generate_steps(wl, min(wl.steps, 4))
    ctx = swam.Swam.from_workload(wl)
    refresh = len(steps)
    assert W.refresh_schedule(len(steps), refresh) == [True] + [False] * (len(steps) - 1)
    compare_schedule(wl, steps, refresh, run_schedule(ctx, wl, steps, refresh))


def test_guided_pair_shares_the_conditional_selection():
    """Two forwards per step (conditional, unconditional): scores and selection come from the conditional one; the
    unconditional context installs that selection and runs its sparse steps with it."""
    swam = _swam()
    wl = small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=2, steps=2)
    kc, ks = wl.budgets
    c0, c1 = W.generate_steps(wl, 2)
    u0, u1 = W.generate_steps(wl.with_(seed=wl.seed + 100), 2)
    cond, uncond = swam.Swam.from_workload(wl), swam.Swam.from_workload(wl)
    out_c, out_u = cond.empty_full().zero_(), uncond.empty_full().zero_()
    cond.step(dev(c0["q"], wl), dev(c0["k"], wl), dev(c0["v"], wl), swam.REFRESH_FULL, out_c)
    uncond.step(dev(u0["q"], wl), dev(u0["k"], wl), dev(u0["v"], wl), swam.REFRESH_FULL, out_u)
    own = [t.clone() for t in uncond.selection()]
    uncond.set_selection(*cond.selection())
    for a, b in zip(uncond.selection(), cond.selection()):
        assert torch.equal(a, b)
    assert not torch.equal(own[0], cond.selection()[0])        # the unconditional forward would have chosen differently
    cond.step(dev(c1["q"], wl), dev(c1["k"], wl), dev(c1["v"], wl), swam.REUSE, out_c)
    uncond.step(dev(u1["q"], wl), dev(u1["k"], wl), dev(u1["v"], wl), swam.REUSE, out_u)
    cond.check()
    uncond.check()
    args = (wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, kc, ks)
    st_c = ora.full_step(ora.StepState(), c0["q"], c0["k"], c0["v"], *args)
    st_u = ora.full_step(ora.StepState(), u0["q"], u0["k"], u0["v"], *args)
    assert np.array_equal(cond.selection()[0].cpu().numpy(), st_c.sel["sel_idx"]), st_c.sel["margins"]
    st_u.pack_map, st_u.inv_map = st_c.pack_map, st_c.inv_map
    ora.sparse_step(st_c, c1["q"], c1["k"], c1["v"])
    ora.sparse_step(st_u, u1["q"], u1["k"], u1["v"])
    check_float(f64(out_c), st_c.out, wl.dtype)
    check_float(f64(out_u), st_u.out, wl.dtype)


def test_exported_state_continues_in_another_context():
    swam = _swam()
    wl = small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=2, steps=3)
    x0, x1, x2 = W.generate_steps(wl, 3)
    a = swam.Swam.from_workload(wl)
    out_a = a.empty_full().zero_()
    with pytest.raises(swam.SwamError) as e:
        a.export_state()
    assert e.value.code == swam.ERR_STATE                      # nothing to export before a refresh
    a.step(dev(x0["q"], wl), dev(x0["k"], wl), dev(x0["v"], wl), swam.REFRESH_FULL, out_a)
    state, out_b = a.export_state(), out_a.clone()
    b = swam.Swam.from_workload(wl)
    b.import_state(state)
    for x in (x1, x2):
        a.step(dev(x["q"], wl), dev(x["k"], wl), dev(x["v"], wl), swam.REUSE, out_a)
        b.step(dev(x["q"], wl), dev(x["k"], wl), dev(x["v"], wl), swam.REUSE, out_b)
    a.check()
    b.check()
    assert torch.equal(out_a, out_b)
    for ta, tb in zip(a.selection() + a.cached_scores(), b.selection() + b.cached_scores()):
        assert torch.equal(ta, tb)
    with pytest.raises(ValueError):
        b.import_state(state[:-1])


@pytest.mark.parametrize("path", ["fused", "kv_gathered_in_kernel"])
def test_corrupt_installed_selection_is_reported_not_followed(path):
    swam = _swam()
    wl = small()
    x0, x1 = W.generate_steps(wl, 2)
    ctx = swam.Swam.from_workload(wl)
    ctx.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_FUSED if path == "fused" else swam.SPARSE_FUSED_KV)
    out = ctx.empty_full().zero_()
    ctx.step(dev(x0["q"], wl), dev(x0["k"], wl), dev(x0["v"], wl), swam.REFRESH_FULL, out)
    before = out.clone()
    sel, pm, im = (t.clone() for t in ctx.selection())
    bad = pm.clone()
    bad[0, 3] = wl.seq_len + 7
    bad[0, 4] = -1
    ctx.set_selection(sel, bad, im)
    ctx.step(dev(x1["q"], wl), dev(x1["k"], wl), dev(x1["v"], wl), swam.REUSE, out)
    with pytest.raises(swam.SwamError) as e:
        ctx.check()
    assert e.value.code == swam.ERR_DEVICE_CHECK
    # rows of the bad entries were left alone, the context still works
    assert torch.equal(out[0, 3], before[0, 3]) and torch.equal(out[0, 4], before[0, 4])
    ctx.set_selection(sel, pm, im)
    ctx.step(dev(x1["q"], wl), dev(x1["k"], wl), dev(x1["v"], wl), swam.REUSE, out)
    ctx.check()


# ------------------------------------------------------------------ grouped-query attention (fewer key/value heads)
GQA_CASES = [
    ("tiny", dict(n_heads=4, n_kv_heads=2)),                                                           # fp32 kernels
    ("single_view", dict(n_obs=70, grid_h=10, grid_w=9, n_heads=6, n_kv_heads=2)),                        # D = 64, tcgen05
    ("larger_imagination", dict(n_obs=40, grid_h=7, grid_w=9, n_heads=4, n_kv_heads=1, batch=2)),         # D = 128, one K/V head
    ("single_view", dict(n_obs=9, grid_h=6, grid_w=6, n_heads=4, n_kv_heads=2, head_dim=32)),             # D = 32, mma.sync
]


@pytest.mark.parametrize("name,kw", GQA_CASES, ids=["f32", "d64", "d128_mqa", "d32"])
def test_grouped_query_stages_match_oracle(name, kw):
    """Score (both normaliser sources), pack and attention with K and V holding fewer heads than Q."""
    swam = _swam()
    wl = W.WORKLOADS[name].with_(**kw)
    x = W.generate_steps(wl, 1)[0]
    assert x["k"].shape[2] == wl.kv_heads and x["q"].shape[2] == wl.n_heads
    ctx = swam.Swam.from_workload(wl)
    q, k, v = (dev(x[n], wl) for n in "qkv")
    out, lse = ctx.sparse_attn(q, k, v, want_lse=True)
    want, wlse = ora.attention(x["q"], x["k"], x["v"])
    check_float(f64(out), want, wl.dtype)
    assert np.abs(lse.cpu().numpy() - wlse).max() <= (1e-4 if wl.dtype == W.F32 else 2e-3)
    lse_act = np.ascontiguousarray(wlse[:, :, wl.seq_len - wl.n_action:]).astype(np.float32)
    s64 = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse_act.astype(np.float64))
    for given in (torch.from_numpy(lse_act).cuda(), None):
        got = ctx.score(q, k, given).cpu().numpy()
        rel = np.abs(got - s64) / np.maximum(s64, 1e-30)
        assert rel.max() <= SCORE_REL, rel.max()
    sel, pm, im = ctx.select(ctx.score(q, k))
    qp, kp, vp = ctx.pack(q, k, v, pm)
    assert kp.shape[2] == wl.kv_heads and qp.shape[2] == wl.n_heads
    pm_np = pm.cpu().numpy()
    for src, gotp in ((x["q"], qp), (x["k"], kp), (x["v"], vp)):
        assert np.array_equal(gotp.float().cpu().numpy(), ora.pack(src, pm_np))
    outp = ctx.sparse_attn(qp, kp, vp)
    wantp, _ = ora.attention(ora.pack(x["q"], pm_np), ora.pack(x["k"], pm_np), ora.pack(x["v"], pm_np))
    check_float(f64(outp), wantp, wl.dtype)
    ctx.check()


@pytest.mark.parametrize("name,kw", GQA_CASES[1:3], ids=["d64", "d128_mqa"])
def test_grouped_query_schedule_matches_oracle(name, kw):
    swam = _swam()
    wl = W.WORKLOADS[name].with_(steps=3, **kw)
    steps = W.generate_steps(wl)
    ctx = swam.Swam.from_workload(wl)
    log = run_schedule(ctx, wl, steps, wl.refresh)
    compare_schedule(wl, steps, wl.refresh, log)
    # the sparse path that gathers key and value rows inside the attention kernel reads the narrower K and V too
    gkv = swam.Swam.from_workload(wl)
    gkv.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_FUSED_KV)
    log_g = run_schedule(gkv, wl, steps, wl.refresh)
    assert all(np.array_equal(a["out"], b["out"]) for a, b in zip(log, log_g))
    # light refresh and the host-buffer path see the narrower K and V as well
    out = ctx.empty_full().zero_()
    x0, x1 = steps[0], steps[1]
    ctx.step(dev(x0["q"], wl), dev(x0["k"], wl), dev(x0["v"], wl), swam.REFRESH_FULL, out)
    ctx.step(dev(x1["q"], wl), dev(x1["k"], wl), dev(x1["v"], wl), swam.REFRESH_LIGHT, out)
    ctx.check()
    tdt = swam.torch_dtype(wl.dtype)
    pinned = [{n: torch.from_numpy(x[n]).to(tdt).pin_memory() for n in "qkv"} for x in (x0, x1)]
    out_h = torch.empty(out.shape, dtype=tdt).pin_memory()
    host_ctx = swam.Swam.from_workload(wl)
    host_ctx.step_host(pinned[0]["q"], pinned[0]["k"], pinned[0]["v"], swam.REFRESH_FULL, out_h)
    host_ctx.step_host(pinned[1]["q"], pinned[1]["k"], pinned[1]["v"], swam.REFRESH_LIGHT, out_h)
    host_ctx.host_join()
    torch.cuda.synchronize()
    host_ctx.check()
    assert torch.equal(out_h.cuda(), out)


@pytest.mark.parametrize("wl", [W.WORKLOADS["tiny"], small(batch=2), small("multi_view", batch=2, n_obs=33, grid_h=5, grid_w=4, n_heads=2)],
                         ids=["f32", "d64", "multiview"])
def test_step_leaves_the_layer_quality_of_its_scores(wl):
    """The (R, E, Q) diagnostics of Eq. 9 that a refresh step caches equal those of the stand-alone scoring call on the
    same scores (the selection kernel computes them in passing) and match the oracle."""
    swam = _swam()
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    out = ctx.empty_full().zero_()
    q, k, v = (dev(x[n], wl) for n in "qkv")
    for mode in (swam.REFRESH_FULL, swam.REFRESH_LIGHT):
        ctx.step(q, k, v, mode, out)
        ctx.check()
        scores, lse, qual = (t.clone() for t in ctx.cached_scores())
        _, qual_alone = ctx.score(q, k, lse if mode == swam.REFRESH_FULL else None, quality=True)
        assert torch.equal(qual, qual_alone)
        want = ora.quality(scores.cpu().numpy())
        assert np.abs(qual.cpu().numpy() - want).max() <= 1e-5 * max(1.0, np.abs(want).max())


# ------------------------------------------------------------------ visibility constraints (segment prefixes)
VIS_CASES = [
    ("tiny", dict()),                                                                           # fp32 kernels
    ("single_view", dict(n_obs=9, grid_h=6, grid_w=6, n_heads=2, head_dim=32)),                  # mma.sync kernel
    ("single_view", dict(n_obs=200, grid_h=10, grid_w=9, n_heads=3)),                            # tcgen05, D = 64
    ("larger_imagination", dict(n_obs=300, grid_h=7, grid_w=9, n_heads=2, batch=2)),             # tcgen05, D = 128
]
VIS_SETTINGS = [(0, 1, 2), (0, 2, 2), (2, 1, 1), (1, 1, 2)]   # what observed / future / action rows see


@pytest.mark.parametrize("name,kw", VIS_CASES, ids=["f32", "d32", "d64", "d128"])
@pytest.mark.parametrize("sees", VIS_SETTINGS, ids=["causal", "obs_isolated", "no_action_keys", "obs_sees_future"])
def test_attention_with_segment_visibility(name, kw, sees):
    swam = _swam()
    wl = W.WORKLOADS[name].with_(**kw)
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    ctx.set_visibility(*sees)
    q, k, v = (dev(x[n], wl) for n in "qkv")
    out, lse = ctx.sparse_attn(q, k, v, want_lse=True)
    ctx.check()
    fut_end = wl.n_obs + wl.n_frames * wl.n_spatial
    want, wlse = ora.attention(x["q"], x["k"], x["v"], visibility=(wl.n_obs, fut_end, sees))
    check_float(f64(out), want, wl.dtype)
    assert np.abs(lse.cpu().numpy() - wlse).max() <= (1e-4 if wl.dtype == W.F32 else 2e-3)
    # the normalisers the scorer computes run over the keys the action rows see
    got = ctx.score(q, k).cpu().numpy()
    s64 = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action,
                    lse=ora.action_lse(x["q"], x["k"], wl.n_action, n_visible=[wl.n_obs, fut_end, wl.seq_len][sees[2]]))
    rel = np.abs(got - s64) / np.maximum(s64, 1e-30)
    assert rel.max() <= SCORE_REL, rel.max()
    # a length that is neither the full nor the packed sequence has no segment boundaries
    with pytest.raises(swam.SwamError) as e:
        ctx.sparse_attn(q[:, :wl.seq_len - 1].contiguous(), k[:, :wl.seq_len - 1].contiguous(), v[:, :wl.seq_len - 1].contiguous())
    assert e.value.code == swam.ERR_UNSUPPORTED


@pytest.mark.parametrize("wl", [
    W.WORKLOADS["tiny"],
    small(batch=2),
    small("larger_imagination", n_obs=140, grid_h=7, grid_w=9, n_heads=2, steps=3),
], ids=["f32", "d64", "d128"])
@pytest.mark.parametrize("sees", [(0, 1, 2), (2, 1, 1)], ids=["causal", "no_action_keys"])
def test_schedule_with_segment_visibility(wl, sees):
    """Full and sparse steps under restricted visibility: the packed sequence has its own segment boundaries."""
    swam = _swam()
    steps = W.generate_steps(wl)
    kc, ks = wl.budgets
    want = ora.run_steps(steps, wl.refresh, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, kc, ks, sees=sees)
    outs = []
    for path in (swam.SPARSE_FUSED, swam.SPARSE_STAGED, swam.SPARSE_FUSED_KV):
        ctx = swam.Swam.from_workload(wl)
        ctx.set_visibility(*sees)
        ctx.set_option(swam.OPT_SPARSE_PATH, path)
        log = run_schedule(ctx, wl, steps, wl.refresh)
        for t, (g, w) in enumerate(zip(log, want)):
            rel = np.abs(g["scores"] - w["scores"].astype(np.float64)) / np.maximum(w["scores"], 1e-30)
            assert rel.max() <= SCORE_REL, (t, rel.max())
            assert np.array_equal(g["sel"], w["sel_idx"]), (t, w["margins"])
            check_float(g["out"], w["out"], wl.dtype)
        outs.append(log[-1]["out"])
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[2], outs[1])


def test_visibility_option_validation():
    swam = _swam()
    ctx = swam.Swam.from_workload(W.WORKLOADS["tiny"])
    for bad in ((0, 0, 2), (2, 2, 0), (3, 2, 2)):
        with pytest.raises(swam.SwamError) as e:
            ctx.set_visibility(*bad)
        assert e.value.code == swam.ERR_INVALID_ARG
    ctx.set_visibility(2, 2, 2)


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_survives():
    """Failure detection without a fault: a one-warp kernel waits, with a limit of 1e5 cycles, on a barrier that
    nothing completes; it returns by itself, swam_check reports the timeout once, and the next calls work."""
    swam = _swam()
    wl = small()
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    q, k, v = (dev(x[n], wl) for n in "qkv")
    out = ctx.empty_full().zero_()
    ctx.step(q, k, v, swam.REFRESH_FULL, out)
    ctx.check()
    before = out.clone()
    ctx.selftest_timeout(100_000)
    with pytest.raises(swam.SwamError) as e:
        ctx.check()
    assert e.value.code == swam.ERR_TIMEOUT and "bounded wait" in str(e.value)
    ctx.check()                                   # the word was cleared: no second report
    ctx.step(q, k, v, swam.REFRESH_FULL, out)     # and the context still computes the same thing
    ctx.check()
    assert torch.equal(out, before)
    with pytest.raises(swam.SwamError) as e:
        ctx.selftest_timeout(0)
    assert e.value.code == swam.ERR_INVALID_ARG


def test_reuse_before_refresh_is_a_state_error():
    swam = _swam()
    wl = W.WORKLOADS["tiny"]
    ctx = swam.Swam.from_workload(wl)
    t = ctx.empty_full().zero_()
    with pytest.raises(swam.SwamError) as e:
        ctx.step(t, t, t, swam.REUSE, ctx.empty_full())
    assert e.value.code == swam.ERR_STATE


def test_host_buffer_step_matches_device_step():
    swam = _swam()
    wl = small()
    steps = W.generate_steps(wl, 2)
    ctx_a, ctx_b = swam.Swam.from_workload(wl), swam.Swam.from_workload(wl)
    out_dev = ctx_a.empty_full()
    out_host = torch.empty(out_dev.shape, dtype=out_dev.dtype).pin_memory()
    for t, x in enumerate(steps):
        mode = swam.REFRESH_FULL if t == 0 else swam.REUSE
        hq, hk, hv = (torch.from_numpy(x[n]).to(out_dev.dtype).pin_memory() for n in "qkv")
        ctx_a.step(hq.cuda(), hk.cuda(), hv.cuda(), mode, out_dev)
        ctx_b.step_host(hq, hk, hv, mode, out_host)
        ctx_b.check()
        assert torch.equal(out_dev.cpu(), out_host)


@pytest.mark.parametrize("rows", ["retained", "all", "pageable"])
def test_host_buffer_steps_pipeline_without_synchronising_in_between(rows):
    """Five calls enqueued back to back; the reuse steps bring only the retained rows across PCIe (the default, from
    pinned buffers), whole tensors on request, and whole tensors when the buffers are pageable: same bits each way."""
    swam = _swam()
    wl = small(steps=5)
    steps = W.generate_steps(wl)
    ctx_a, ctx_b = swam.Swam.from_workload(wl), swam.Swam.from_workload(wl)
    out_dev = ctx_a.empty_full()
    tdt = out_dev.dtype
    pin = (lambda t: t) if rows == "pageable" else (lambda t: t.pin_memory())
    host_in = [[pin(torch.from_numpy(x[n]).to(tdt)) for n in "qkv"] for x in steps]
    host_out = [torch.empty(out_dev.shape, dtype=tdt).pin_memory() for _ in steps]
    if rows == "all":
        ctx_b.set_option(swam.OPT_HOST_ROWS, swam.HOST_ROWS_ALL)
    want = []
    for t, (hq, hk, hv) in enumerate(host_in):
        mode = swam.REFRESH_FULL if t % 2 == 0 else swam.REUSE
        ctx_a.step(hq.cuda(), hk.cuda(), hv.cuda(), mode, out_dev)
        want.append(out_dev.cpu().clone())
    for t, (hq, hk, hv) in enumerate(host_in):          # five calls enqueued back to back
        ctx_b.step_host(hq, hk, hv, swam.REFRESH_FULL if t % 2 == 0 else swam.REUSE, host_out[t])
    ctx_b.check()
    for t in range(len(steps)):
        assert torch.equal(want[t], host_out[t]), t


# ------------------------------------------------------------------ several profiled layers (Eq. 3, Eq. 9, Eq. 11)
@pytest.mark.parametrize("wl,n_layers,k_layer", [
    (small(batch=2), 5, 2),
    (small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=2), 6, 6),
], ids=["5_layers_top2", "6_layers_all"])
def test_multi_layer_aggregation_and_selection(wl, n_layers, k_layer):
    swam = _swam()
    layers = W.generate_steps(wl.with_(rho=0.5), n_layers)          # one (q, k) pair per profiled layer
    ctx = swam.Swam.from_workload(wl)
    kc, ks = wl.budgets
    s_dev, q_dev = [], []
    for x in layers:
        s, qual = ctx.score(dev(x["q"], wl), dev(x["k"], wl), quality=True)
        s_dev.append(s)
        q_dev.append(qual)
    ls, lq = torch.stack(s_dev).contiguous(), torch.stack(q_dev).contiguous()
    v_core, v_all, core_layers = ctx.aggregate(ls, lq, k_layer)
    sel, pm, im = ctx.select_maps(v_core, v_all)
    ctx.check()
    # stage-isolated: the oracle on the device's own per-layer arrays must agree bit for bit
    wc, wa, wl_layers = ora.aggregate(ls.cpu().numpy(), lq.cpu().numpy(), k_layer)
    assert np.array_equal(core_layers.cpu().numpy(), wl_layers)
    assert np.array_equal(v_core.cpu().numpy(), wc) and np.array_equal(v_all.cpu().numpy(), wa)
    want_sel = ora.select2(wc, wa, kc, ks)
    wpm, wim = ora.maps(want_sel, wl.n_obs, wl.n_spatial, wl.n_action)
    assert np.array_equal(sel.cpu().numpy(), want_sel)
    assert np.array_equal(pm.cpu().numpy(), wpm) and np.array_equal(im.cpu().numpy(), wim)
    # end to end from the oracle's own scores and qualities
    os_ = np.stack([ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action).astype(np.float32)
                    for x in layers])
    oq = np.stack([ora.quality(s) for s in os_]).astype(np.float32)
    ec, ea, el = ora.aggregate(os_, oq, k_layer)
    assert np.array_equal(el, wl_layers)
    assert (np.abs(v_core.cpu().numpy() - ec) / ec).max() <= 1e-4 and (np.abs(v_all.cpu().numpy() - ea) / ea).max() <= 1e-4
    if k_layer == n_layers:
        assert torch.equal(v_core, v_all)


def test_single_layer_aggregation_is_identity():
    swam = _swam()
    wl = small()
    x = W.generate_steps(wl, 1)[0]
    ctx = swam.Swam.from_workload(wl)
    s, qual = ctx.score(dev(x["q"], wl), dev(x["k"], wl), quality=True)
    v_core, v_all, _ = ctx.aggregate(s.unsqueeze(0).contiguous(), qual.unsqueeze(0).contiguous(), 1)
    assert torch.equal(v_core, s) and torch.equal(v_all, s)
    a = ctx.select(s)
    b = ctx.select_maps(v_core, v_all)
    for t, u in zip(a, b):
        assert torch.equal(t, u)


# ------------------------------------------------------------------ more edge cases
def test_cycle_replayed_from_a_cuda_graph_equals_eager():
    """The step has a fixed shape, so a refresh cycle can be captured once and replayed (what bench.py times)."""
    swam = _swam()
    wl = small(batch=2)
    steps = W.generate_steps(wl, 2)
    d = [{n: dev(x[n], wl) for n in "qkv"} for x in steps]
    eager, graphed = swam.Swam.from_workload(wl), swam.Swam.from_workload(wl)
    out_e, out_g = eager.empty_full().zero_(), graphed.empty_full().zero_()

    def cycle(ctx, out):
        ctx.step(d[0]["q"], d[0]["k"], d[0]["v"], swam.REFRESH_FULL, out)
        ctx.step(d[1]["q"], d[1]["k"], d[1]["v"], swam.REUSE, out)

    cycle(eager, out_e)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        cycle(graphed, out_g)                      # warm-up outside capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    out_g.zero_()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        cycle(graphed, out_g)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    graphed.check()
    assert torch.equal(out_e, out_g)
    for a, b in zip(eager.selection(), graphed.selection()):
        assert torch.equal(a, b)


def test_sweep_tool_reports_consistent_numbers_on_a_small_shape():
    """The keep-ratio x refresh-interval sweep tool on a small shape: every key of its record is there, the overlap
    measures lie in [0, 1], and keeping every token reproduces the dense output."""
    swam = _swam()
    from paper_2609_38984_b200 import sweep
    base = small("larger_imagination", n_obs=40, grid_h=7, grid_w=9, n_heads=2, steps=4, seed=4)
    n_steps = 4
    host = W.generate_steps(base, n_steps)
    dev_steps = [{n: dev(x[n], base) for n in "qkv"} for x in host]
    dense_ctx = swam.Swam.from_workload(base)
    dense_outs = [dense_ctx.sparse_attn(x["q"], x["k"], x["v"]) for x in dev_steps]
    for keep, refresh in ((0.3, 2), (1.0, 2), (0.5, 1), (0.2, 4)):
        wl = W.variant_workload(base.with_(keep=keep, k_core=None, k_anchor=None), "combined").with_(steps=n_steps, refresh=refresh)
        rec = sweep.run_config(wl, refresh, n_steps, dev_steps, dense_outs)
        for key in ("shape", "variant", "keep", "refresh", "k_core", "k_anchor", "packed_len", "steps", "full_steps", "stage_us",
                    "full_step_us", "sparse_step_us", "schedule_us", "schedule_graph_us", "tokens_per_s",
                    "iou_consecutive_steps", "overlap_eq13_consecutive_steps", "rel_l2_vs_dense_per_step"):
            assert key in rec, key
        assert sorted(rec["stage_us"]) == ["attn_dense", "attn_packed", "pack", "scatter", "score", "select"]
        assert all(v > 0 for v in rec["stage_us"].values()) and rec["tokens_per_s"] > 0 and rec["schedule_graph_us"] > 0
        assert rec["full_steps"] == len([t for t in range(n_steps) if t % refresh == 0])
        assert rec["packed_len"] == wl.packed_len and rec["k_core"] + rec["k_anchor"] == wl.k_keep
        assert 0.0 <= rec["iou_consecutive_steps"] <= 1.0 and 0.0 <= rec["overlap_eq13_consecutive_steps"] <= 1.0
        assert len(rec["rel_l2_vs_dense_per_step"]) == n_steps
        if keep == 1.0 or refresh == 1:
            # every token kept, or every step dense: the output is the dense output (up to the kernel's own
            # run-to-run identical arithmetic: same kernel, same inputs)
            assert max(rec["rel_l2_vs_dense_per_step"]) <= 1e-6, rec["rel_l2_vs_dense_per_step"]
        else:
            assert rec["rel_l2_vs_dense_per_step"][0] <= 1e-6          # step 0 is a full step


def test_keep_nothing_leaves_only_observed_and_action_rows():
    swam = _swam()
    wl = small(k_core=0, k_anchor=0)
    assert wl.packed_len == wl.n_obs + wl.n_action
    steps = W.generate_steps(wl, 2)
    ctx = swam.Swam.from_workload(wl)
    compare_schedule(wl, steps, 2, run_schedule(ctx, wl, steps, 2))
    _, pm, im = ctx.selection()
    L = wl.seq_len
    assert pm.cpu().numpy()[0].tolist() == list(range(wl.n_obs)) + list(range(L - wl.n_action, L))
    assert int((im < 0).sum()) == wl.batch * wl.n_frames * wl.n_spatial
