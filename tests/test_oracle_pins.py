"""Pins the CPU oracle to facts fixed by the paper and by mathematics (no GPU).

Each test is chosen so that a plausible mistake in the oracle (a dropped term,
a wrong sign or index, a transposed operand, a wrong tie-break) fails it.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import reference as ora
from paper_2609_38984_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_qkv(seed, b, n, nh, d):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((b, n, nh, d)).astype(np.float32) for _ in range(3)]


# ------------------------------------------------------------------ attention
def test_attention_matches_library_fp64():
    q, k, v = _rand_qkv(0, 2, 37, 3, 16)
    out, lse = ora.attention(q, k, v)
    tq, tk, tv = [torch.from_numpy(x).double().permute(0, 2, 1, 3) for x in (q, k, v)]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    assert np.abs(out - ref).max() < 1e-12
    logits = torch.einsum("bhqd,bhkd->bhqk", tq, tk) / np.sqrt(16)
    assert np.abs(lse - torch.logsumexp(logits, -1).numpy()).max() < 1e-12


def test_grouped_query_attention_matches_library_head_mapping():
    """K and V with fewer heads: query head h reads head h // (N_h / N_kv), as the library's own grouped-query
    attention does; a head order of "h % N_kv" (the plausible mistake) gives a different answer."""
    rng = np.random.default_rng(11)
    q = rng.standard_normal((2, 23, 6, 8)).astype(np.float32)
    k = rng.standard_normal((2, 23, 2, 8)).astype(np.float32)
    v = rng.standard_normal((2, 23, 2, 8)).astype(np.float32)
    out, _ = ora.attention(q, k, v)
    tq, tk, tv = [torch.from_numpy(x).double().permute(0, 2, 1, 3) for x in (q, k, v)]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, enable_gqa=True).permute(0, 2, 1, 3).numpy()
    assert np.abs(out - ref).max() < 1e-12
    wrong = torch.nn.functional.scaled_dot_product_attention(tq, tk.repeat(1, 3, 1, 1), tv.repeat(1, 3, 1, 1))
    assert np.abs(out - wrong.permute(0, 2, 1, 3).numpy()).max() > 1e-3
    # the score sees the same mapping: expanding the key heads by hand changes nothing
    s1 = ora.score(q, k, 3, 2, 6, 8)
    s2 = ora.score(q, np.repeat(k, 3, axis=2), 3, 2, 6, 8)
    assert np.array_equal(s1, s2)


def test_attention_scale_and_transpose_sensitivity():
    # non-square: queries from one tensor, keys from another with different statistics; a swapped
    # operand or a missing scale changes the answer
    q, k, v = _rand_qkv(1, 1, 19, 2, 8)
    k *= 3.0
    out, _ = ora.attention(q, k, v, scale=0.25)
    tq, tk, tv = [torch.from_numpy(x).double().permute(0, 2, 1, 3) for x in (q, k, v)]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.25).permute(0, 2, 1, 3).numpy()
    assert np.abs(out - ref).max() < 1e-12


def test_attention_closed_forms():
    q, k, v = _rand_qkv(2, 1, 11, 2, 8)
    # constant values -> constant output
    vc = np.ones_like(v) * 2.5
    out, _ = ora.attention(q, k, vc)
    assert np.abs(out - 2.5).max() < 1e-13
    # a single key -> output equals its value, lse equals the logit
    out1, lse1 = ora.attention_rows(q[:, :1], k[:, :1], v[:, :1], np.array([[0, 0]]))
    assert np.abs(out1[0] - v[0, 0]).max() < 1e-13
    assert np.abs(lse1[0] - (q[0, 0].astype(np.float64) * k[0, 0]).sum(-1) / np.sqrt(8)).max() < 1e-13
    # permuting keys together with values leaves the output unchanged
    perm = np.random.default_rng(3).permutation(11)
    out_a, lse_a = ora.attention(q, k, v)
    out_b, lse_b = ora.attention(q, k[:, perm], v[:, perm])
    assert np.abs(out_a - out_b).max() < 1e-12 and np.abs(lse_a - lse_b).max() < 1e-12
    # zero queries -> uniform weights -> output is the mean value, lse = log n
    out0, lse0 = ora.attention(np.zeros_like(q), k, v)
    assert np.abs(out0 - v.astype(np.float64).mean(1, keepdims=True)).max() < 1e-13
    assert np.abs(lse0 - np.log(11)).max() < 1e-13


def test_attention_rows_subset_equals_full():
    q, k, v = _rand_qkv(4, 2, 23, 2, 8)
    out, lse = ora.attention(q, k, v)
    rows = np.array([[1, 5], [0, 22], [1, 0]])
    o, l = ora.attention_rows(q, k, v, rows)
    for i, (b, r) in enumerate(rows):
        assert np.array_equal(o[i], out[b, r]) and np.array_equal(l[i], lse[b, :, r])


# ------------------------------------------------------------------ weights
def test_query_weights_match_paper_values():
    with open(os.path.join(GOLDEN, "query_weights.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            g, vals = line.split(":")
            want = np.array([float(Fraction(t)) for t in vals.split()])
            got = ora.query_weights(int(g))
            assert got.shape == want.shape and np.abs(got - want).max() < 1e-15
            assert abs(got.sum() - 1.0) < 1e-15
    with pytest.raises(ValueError):
        ora.query_weights(6)


# ------------------------------------------------------------------ score
def _shape():
    return dict(n_obs=5, n_frames=3, n_spatial=7, n_action=12)


def test_score_zero_queries_closed_form():
    sh = _shape()
    L = sh["n_obs"] + sh["n_frames"] * sh["n_spatial"] + sh["n_action"]
    q, k, _ = _rand_qkv(5, 2, L, 3, 8)
    s = ora.score(np.zeros_like(q), k, **sh)
    # every attention weight is 1/L, the weights alpha sum to one, the head average keeps 1/L
    assert np.abs(s - 1.0 / L).max() < 1e-15
    rq = ora.quality(s.astype(np.float32))
    assert np.allclose(rq[:, 0], sh["n_spatial"] / L, rtol=1e-6)     # R = N_s / L
    assert np.allclose(rq[:, 1], 1.0, atol=1e-6)                      # uniform -> entropy 1
    assert np.allclose(rq[:, 2], 0.0, atol=1e-6)


def test_score_equals_full_softmax_definition():
    """Eq. 12 must agree with Eq. 1 + Eq. 2 evaluated from the full H x L attention matrix."""
    sh = _shape()
    n_obs, F, N, H = sh["n_obs"], sh["n_frames"], sh["n_spatial"], sh["n_action"]
    L = n_obs + F * N + H
    nh, d = 3, 8
    q, k, _ = _rand_qkv(6, 2, L, nh, d)
    s = ora.score(q, k, **sh)
    g = H // F
    alpha = np.array([1, 2, 2, 1], dtype=np.float64) / 6.0
    q64, k64 = q.astype(np.float64), k.astype(np.float64)
    for b in range(2):
        logits = np.einsum("ihd,chd->hic", q64[b, L - H:], k64[b]) / np.sqrt(d)     # [h, i, c]
        a = np.exp(logits - logits.max(-1, keepdims=True))
        a /= a.sum(-1, keepdims=True)                                               # softmax over ALL keys
        u = a.mean(0)                                                               # Eq. 1: head average [i, c]
        for f in range(F):
            want = np.zeros(N)
            for t in range(g):
                want += alpha[t] * u[f * g + t, n_obs + f * N: n_obs + (f + 1) * N]  # Eq. 2
            assert np.abs(s[b, f] - want).max() < 1e-14
    # attention mass: 0 < R <= 1 because the normaliser covers all keys
    rq = ora.quality(s.astype(np.float32))
    assert np.all(rq[:, 0] > 0) and np.all(rq[:, 0] <= 1.0)


def test_score_uses_aligned_group_only():
    """Changing an action query of another group must not change frame f's scores."""
    sh = _shape()
    L = sh["n_obs"] + sh["n_frames"] * sh["n_spatial"] + sh["n_action"]
    q, k, _ = _rand_qkv(7, 1, L, 2, 8)
    lse = ora.action_lse(q, k, sh["n_action"])
    s0 = ora.score(q, k, lse=lse, **sh)
    q2 = q.copy()
    q2[0, L - sh["n_action"] + 0] += 1.0          # query 0 belongs to frame 0's group
    lse2 = ora.action_lse(q2, k, sh["n_action"])
    s1 = ora.score(q2, k, lse=lse2, **sh)
    assert not np.allclose(s0[0, 0], s1[0, 0])
    assert np.array_equal(s0[0, 1:], s1[0, 1:])


def test_quality_one_hot_has_zero_entropy():
    s = np.zeros((1, 3, 9), np.float32)
    s[0, 0, 2] = s[0, 1, 4] = s[0, 2, 0] = 0.125
    rq = ora.quality(s)
    assert abs(rq[0, 1]) < 1e-15 and abs(rq[0, 0] - 0.125) < 1e-15 and abs(rq[0, 2] - 0.125) < 1e-15


# ------------------------------------------------------------------ selection
def _brute_topk(keys, cand, n):
    cand = np.asarray(cand)
    order = np.argsort(-keys[cand], kind="stable")      # stable: equal keys keep ascending index order
    return set(cand[order[:n]].tolist())


def _brute_select(s, kc, ks, beta=1.0):
    F, N = s.shape
    pool = _brute_topk(s.max(0).astype(np.float64), np.arange(N), N - ks)
    cores = [_brute_topk(s[f].astype(np.float64), sorted(pool), kc) for f in range(F)]
    rest = sorted(set(range(N)) - set().union(*cores)) if cores else list(range(N))
    s64 = s.astype(np.float64)
    mu = s64.mean(0)
    sd = s64.std(0)
    cv = np.where(mu > 0, sd / np.where(mu > 0, mu, 1.0), 0.0)
    key = mu / (1.0 + beta * cv)
    anchors = _brute_topk(key, rest, ks)
    return pool, cores, anchors, [sorted(c | anchors) for c in cores]


@pytest.mark.parametrize("seed,ties", [(0, False), (1, True), (2, True), (3, False)])
def test_select_matches_brute_force_sort(seed, ties):
    F, N, kc, ks = 4, 48, 9, 13
    s = W.random_scores(seed, 3, F, N, ties=ties)
    res = ora.select(s, kc, ks)
    for b in range(3):
        pool, cores, anchors, ret = _brute_select(s[b], kc, ks)
        assert set(np.nonzero(res["pool"][b])[0].tolist()) == pool
        for f in range(F):
            assert set(np.nonzero(res["core"][b, f])[0].tolist()) == cores[f]
            assert res["sel_idx"][b, f].tolist() == ret[f]
        assert set(res["anchors"][b].tolist()) == anchors


def test_select_guarantees():
    F, N, kc, ks = 5, 64, 14, 18
    s = W.random_scores(11, 4, F, N, ties=True)
    res = ora.select(s, kc, ks)
    for b in range(4):
        pool = res["pool"][b].astype(bool)
        assert pool.sum() == N - ks                                    # |P| = N_s - K_s
        union = np.zeros(N, bool)
        for f in range(F):
            core = res["core"][b, f].astype(bool)
            assert core.sum() == kc and not np.any(core & ~pool)       # C_f within P
            union |= core
        assert (~union).sum() >= ks                                    # |E| >= K_s
        anchors = res["anchors"][b]
        assert len(set(anchors.tolist())) == ks and not np.any(union[anchors])   # anchors within E
        for f in range(F):
            sel = res["sel_idx"][b, f]
            assert len(sel) == kc + ks and np.all(np.diff(sel) > 0)    # exactly K, ascending
            assert set(sel.tolist()) == set(np.nonzero(res["core"][b, f])[0].tolist()) | set(anchors.tolist())


def test_select_all_equal_scores_pins_tie_break():
    F, N, kc, ks = 3, 20, 4, 6
    s = np.full((1, F, N), 0.01, np.float32)
    res = ora.select(s, kc, ks)
    assert np.nonzero(res["pool"][0])[0].tolist() == list(range(N - ks))
    for f in range(F):
        assert np.nonzero(res["core"][0, f])[0].tolist() == list(range(kc))
        assert res["sel_idx"][0, f].tolist() == list(range(kc + ks))
    assert res["anchors"][0].tolist() == list(range(kc, kc + ks))


def test_select_degenerate_budgets():
    F, N = 3, 16
    s = W.random_scores(5, 1, F, N)
    # no anchors: plain per-frame top-K_c
    res = ora.select(s, 5, 0)
    for f in range(F):
        want = sorted(np.argsort(-s[0, f], kind="stable")[:5].tolist())
        assert res["sel_idx"][0, f].tolist() == want
    # keep everything
    res = ora.select(s, 7, 9)
    for f in range(F):
        assert res["sel_idx"][0, f].tolist() == list(range(N))
    # identical frames: CV = 0, anchors are the best mean scores outside the cores
    s_same = np.repeat(s[:, :1], F, axis=1)
    res = ora.select(s_same, 4, 5)
    order = np.argsort(-s_same[0, 0], kind="stable")
    assert set(np.nonzero(res["core"][0, 0])[0].tolist()) == set(order[:4].tolist())
    assert set(res["anchors"][0].tolist()) == set(order[4:9].tolist())
    assert np.array_equal(res["anchor_key"][0], s_same[0, 0].astype(np.float64))


def test_anchor_key_penalises_variation():
    # two positions with the same mean; the one that varies across frames must rank lower
    s = np.zeros((1, 2, 6), np.float32)
    s[0, :, 0] = [0.9, 0.9]            # core in both frames
    s[0, :, 1] = [0.4, 0.4]            # steady
    s[0, :, 2] = [0.7, 0.1]            # same mean 0.4, varying
    s[0, :, 3] = [0.05, 0.05]
    res = ora.select(s, 1, 1)
    key = res["anchor_key"][0]
    assert abs(key[1] - 0.4) < 1e-7
    assert abs(key[2] - 0.4 / (1 + 0.3 / 0.4)) < 1e-7       # std 0.3 (population), mean 0.4
    # position 2 is the core of neither frame? frame 0 core = 0, frame 1 core = 0 -> anchors from {1..5}
    assert res["anchors"][0].tolist() == [1]


def test_budget_rule_against_paper_ratios():
    with open(os.path.join(GOLDEN, "budgets.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            t = line.split()
            if t[0] == "ratio":
                pct, n, k = float(t[1]), int(t[2]), int(t[3])
                assert round(100 * (1 - k / n), 2) == pct
                kc, ks = W.budgets_from_keep(1 - pct / 100, n)
                assert kc + ks == k
            elif t[0] == "queries":
                # App. B.2's query groups: the printed weights exist for exactly these group sizes
                assert int(t[2]) == 32 and len(ora.query_weights(int(t[3]))) == int(t[3])
            else:
                n, kc, ks, k = map(int, t[1:])
                assert kc + ks == k <= n
                if t[0] == "cosmos3_nano":
                    assert W.budgets_from_keep(k / n, n) == (kc, ks)      # the 80:104 split
    # the shapes the benchmark is quoted on
    want = {"tiny": (14, 18), "single_view": (63, 81), "larger_imagination": (133, 174), "multi_view": (188, 244)}
    for name, b in want.items():
        assert W.WORKLOADS[name].budgets == b
    assert [W.sweep_workload(kp, 2).k_keep for kp in W.SWEEP_KEEPS] == [102, 205, 307, 512, 1024]


# ------------------------------------------------------------------ maps, pack, scatter
def test_maps_properties():
    F, N, kc, ks, n_obs, H = 3, 32, 5, 7, 6, 9
    s = W.random_scores(8, 2, F, N)
    sel = ora.select(s, kc, ks)["sel_idx"]
    pack, inv = ora.maps(sel, n_obs, N, H)
    L, Lp = n_obs + F * N + H, n_obs + F * (kc + ks) + H
    assert pack.shape == (2, Lp) and inv.shape == (2, L)
    for b in range(2):
        assert np.all(np.diff(pack[b]) > 0)
        assert np.array_equal(inv[b][pack[b]], np.arange(Lp))
        assert (inv[b] >= 0).sum() == Lp
        assert pack[b][:n_obs].tolist() == list(range(n_obs))
        assert pack[b][-H:].tolist() == list(range(L - H, L))
        for f in range(F):
            seg = pack[b][n_obs + f * (kc + ks): n_obs + (f + 1) * (kc + ks)]
            assert np.array_equal(seg - n_obs - f * N, sel[b, f])
    # keeping everything gives the identity map
    sel_all = ora.select(s, 12, 20)["sel_idx"]
    pack, inv = ora.maps(sel_all, n_obs, N, H)
    assert np.array_equal(pack[0], np.arange(L)) and np.array_equal(inv[0], np.arange(L))


def test_pack_then_scatter_is_identity_on_retained_rows():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((2, 30, 2, 4))
    pm = np.stack([np.sort(rng.choice(30, 11, replace=False)) for _ in range(2)]).astype(np.int32)
    cached = rng.standard_normal(x.shape)
    out = ora.scatter(ora.pack(x, pm), pm, cached)
    for b in range(2):
        keep = np.zeros(30, bool)
        keep[pm[b]] = True
        assert np.array_equal(out[b][keep], x[b][keep])
        assert np.array_equal(out[b][~keep], cached[b][~keep])


# ------------------------------------------------------------------ step loop
def _tiny_steps():
    wl = W.WORKLOADS["tiny"]
    return wl, W.generate_steps(wl)


def test_keep_ratio_one_reproduces_dense_attention():
    wl, steps = _tiny_steps()
    log = ora.run_steps(steps, 2, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, 28, 36)
    for t, x in enumerate(steps):
        dense, _ = ora.attention(x["q"], x["k"], x["v"])
        assert np.array_equal(log[t]["out"], dense)
        assert np.array_equal(log[t]["pack_map"][0], np.arange(wl.seq_len))


def test_refresh_every_step_equals_recomputation():
    wl, steps = _tiny_steps()
    kc, ks = wl.budgets
    log = ora.run_steps(steps, 1, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, kc, ks)
    for t, x in enumerate(steps):
        fresh = ora.full_step(ora.StepState(), x["q"], x["k"], x["v"], wl.n_obs, wl.n_frames, wl.n_spatial,
                              wl.n_action, kc, ks)
        assert np.array_equal(log[t]["sel_idx"], fresh.sel["sel_idx"])
        assert np.array_equal(log[t]["out"], fresh.out)
        dense, _ = ora.attention(x["q"], x["k"], x["v"])
        assert np.array_equal(log[t]["out"], dense)


def test_sparse_step_semantics():
    wl, steps = _tiny_steps()
    kc, ks = wl.budgets
    log = ora.run_steps(steps, 2, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, kc, ks)
    assert [e["full"] for e in log] == [True, False, True]
    pm, inv = log[1]["pack_map"][0], log[1]["inv_map"][0]
    omitted = inv < 0
    assert omitted.sum() == wl.seq_len - wl.packed_len
    assert not omitted[:wl.n_obs].any() and not omitted[-wl.n_action:].any()
    # omitted rows keep the last full step's values exactly; retained rows are the packed attention
    assert np.array_equal(log[1]["out"][0][omitted], log[0]["out"][0][omitted])
    x = steps[1]
    op, _ = ora.attention(ora.pack(x["q"], log[1]["pack_map"]), ora.pack(x["k"], log[1]["pack_map"]),
                          ora.pack(x["v"], log[1]["pack_map"]))
    assert np.array_equal(log[1]["out"][0][pm], op[0])
    # the selection is reused, not recomputed, on the sparse step
    assert np.array_equal(log[1]["sel_idx"], log[0]["sel_idx"])


def test_overlap_measure():
    p = np.array([0.2, 0.3, 0.5])
    assert abs(ora.overlap(p, p * 7) - 1.0) < 1e-15
    assert ora.overlap(np.array([1.0, 0, 0]), np.array([0, 2.0, 1.0])) == 0.0
    assert abs(ora.overlap(np.array([1.0, 1.0]), np.array([3.0, 1.0])) - 0.75) < 1e-15


# ------------------------------------------------------------------ multi-layer aggregation (Eq. 3, Eq. 9, Eq. 11)
def _layers(seed, nl, b, f, n):
    s = np.stack([W.random_scores(seed + l, b, f, n) for l in range(nl)])
    q = np.stack([ora.quality(s[l]) for l in range(nl)]).astype(np.float32)
    return s, q


def test_aggregate_single_layer_is_the_layer_itself():
    s, q = _layers(40, 1, 2, 3, 17)
    vc, va, layers = ora.aggregate(s, q, 1)
    assert np.array_equal(vc, s[0]) and np.array_equal(va, s[0]) and layers.tolist() == [[0], [0]]
    # and the selection from (V, V_all) equals the single-map selection
    assert np.array_equal(ora.select2(vc, va, 4, 5), ora.select(s[0], 4, 5)["sel_idx"])


def test_aggregate_against_direct_weighted_mean():
    nl, b, f, n, kl = 5, 2, 3, 19, 2
    s, q = _layers(50, nl, b, f, n)
    q[:, :, 2] = np.array([[0.1, 0.4], [0.5, 0.2], [0.3, 0.6], [0.05, 0.1], [0.5, 0.3]], np.float32)   # with a tie in sample 0
    vc, va, layers = ora.aggregate(s, q, kl)
    assert layers.tolist() == [[1, 4], [0, 2]]                      # top-2 by Q (sample 0: the 0.5/0.5 tie beats 0.3)
    for i in range(b):
        w = q[:, i, 2].astype(np.float64)
        want_all = np.tensordot(w, s[:, i].astype(np.float64), axes=1) / w.sum()
        sel = layers[i]
        want_core = np.tensordot(w[sel], s[sel, i].astype(np.float64), axes=1) / w[sel].sum()
        # results are stored as fp32: half an ulp at these magnitudes is below 4e-9
        assert np.abs(va[i] - want_all).max() <= 5e-9 and np.abs(vc[i] - want_core).max() <= 5e-9
    # all layers selected: V equals V_all
    vc2, va2, _ = ora.aggregate(s, q, nl)
    assert np.array_equal(vc2, va2)
    # equal qualities: plain mean over layers; zero qualities fall back to the plain mean as well
    q[:, :, 2] = 0.25
    _, va3, _ = ora.aggregate(s, q, nl)
    assert np.abs(va3 - s.astype(np.float64).mean(0)).max() <= 5e-9
    q[:, :, 2] = 0.0
    _, va4, _ = ora.aggregate(s, q, nl)
    assert np.abs(va4 - s.astype(np.float64).mean(0)).max() <= 5e-9


def test_select2_uses_core_map_for_cores_and_all_map_for_anchors():
    f, n, kc, ks = 2, 12, 2, 3
    v_core = np.zeros((1, f, n), np.float32)
    v_all = np.zeros((1, f, n), np.float32)
    v_core[0, 0, [3, 7]] = [0.9, 0.8]          # frame 0 cores
    v_core[0, 1, [5, 1]] = [0.9, 0.7]          # frame 1 cores
    v_all[0, :, 10] = 0.5                      # strong and steady in V_all only
    v_all[0, :, 11] = 0.4
    v_all[0, :, 2] = 0.3
    v_all[0, :, 3] = 0.95                      # core position: must not become an anchor
    sel = ora.select2(v_core, v_all, kc, ks)
    assert sel[0, 0].tolist() == [2, 3, 7, 10, 11] and sel[0, 1].tolist() == [1, 2, 5, 10, 11]



def test_segment_prefix_visibility_matches_library_mask():
    """Rows restricted to a key prefix per segment equal the library's attention under the corresponding boolean mask;
    a mask transposed (keys restricted by their own segment instead of the query's) gives a different answer."""
    q, k, v = _rand_qkv(5, 2, 29, 2, 8)
    obs_end, fut_end, n = 7, 21, 29
    for sees in ((0, 1, 2), (2, 1, 2), (0, 2, 1), (2, 2, 2)):
        out, lse = ora.attention(q, k, v, visibility=(obs_end, fut_end, sees))
        ends = np.array([obs_end, fut_end, n])
        seg = (np.arange(n) >= obs_end).astype(int) + (np.arange(n) >= fut_end).astype(int)
        mask = np.arange(n)[None, :] < ends[np.array(sees)[seg]][:, None]            # [query, key]
        tq, tk, tv = [torch.from_numpy(x).double().permute(0, 2, 1, 3) for x in (q, k, v)]
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask))
        assert np.abs(out - ref.permute(0, 2, 1, 3).numpy()).max() < 1e-12
        logits = torch.einsum("bhqd,bhkd->bhqk", tq, tk) / np.sqrt(8)
        logits = logits.masked_fill(~torch.from_numpy(mask), -np.inf)
        assert np.abs(lse - torch.logsumexp(logits, -1).numpy()).max() < 1e-12
        if sees != (2, 2, 2):
            wrong = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask.T.copy() | np.eye(n, dtype=bool)))
            assert np.abs(out - wrong.permute(0, 2, 1, 3).numpy()).max() > 1e-3
    # the action-row normaliser over a key prefix is the masked log-sum-exp of those rows
    lam = ora.action_lse(q, k, 8, n_visible=fut_end)
    _, lse_vis = ora.attention(q, k, v, visibility=(obs_end, fut_end, (2, 2, 1)))
    assert np.abs(lam - lse_vis[:, :, n - 8:]).max() < 1e-12
