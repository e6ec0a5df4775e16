"""Whole denoising schedules at the benchmark's full sizes against the oracle (Sec. 4.2's full / sparse loop, Eq. 7).

Coverage rule: at every step of the schedule the scores (every element), the selected indices, the pack map and the
inverse map (bit-exact, both stage-isolated on the device's own score array and end to end on the oracle's), and the
omitted rows (bit-exact against the previous step's output) are checked.  Attention outputs are compared with the
oracle on EVERY row for the first full and the first sparse step (of every sample at the larger-imagination shape and
the single-view shape, of one of the eight samples at the multi-view shape) and on at least 512 seeded (sample, row)
pairs for each later step, which always include every action row and the first and last row of every 128-row tile.
The single-view shape compares every row at every step.  Refresh intervals 1 and 4 run at the sweep shape (seed 4).
"""
import numpy as np
import pytest
import torch

from oracle import reference as ora
from paper_2609_38984_b200 import workloads as W

pytestmark = pytest.mark.gpu

SCORE_REL = 1e-5   # relative error of a score (measured maxima: below 1e-6 at every benchmark shape)
TILE = 128


def all_rows(batches, n):
    return np.stack(np.meshgrid(np.asarray(batches), np.arange(n), indexing="ij"), axis=-1).reshape(-1, 2).astype(np.int32)


def sampled_rows(rng, batch, n, n_action, n_pairs):
    """Seeded (sample, row) pairs: every action row of every sample, the first and last row of each 128-row tile
    (a seeded sample each), then random pairs up to n_pairs."""
    rows = {(b, r) for b in range(batch) for r in range(n - n_action, n)}
    for t0 in range(0, n, TILE):
        rows.add((int(rng.integers(0, batch)), t0))
        rows.add((int(rng.integers(0, batch)), min(t0 + TILE, n) - 1))
    while len(rows) < n_pairs:
        rows.add((int(rng.integers(0, batch)), int(rng.integers(0, n))))
    return np.array(sorted(rows), dtype=np.int32)


def check_bf16(got, want, what):
    err = np.abs(got - want)
    assert err.max() <= 2e-2, (what, err.max())
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= 1e-2, (what, rel)


def run_schedule_against_oracle(wl, refresh, n_steps, every_row, n_pairs=512, every_row_steps=2):
    """every_row: "all" (every sample), an int (that sample), or None; applies to the first `every_row_steps` steps
    (with refresh 2: the first full and the first sparse step).  Returns the largest relative score error seen."""
    from paper_2609_38984_b200 import swam
    kc, ks = wl.budgets
    B, L, Lp, H = wl.batch, wl.seq_len, wl.packed_len, wl.n_action
    gen = W.Generator(wl)
    ctx = swam.Swam.from_workload(wl)
    out = ctx.empty_full().zero_()
    rng = np.random.default_rng(1000 + wl.seed)
    sched = W.refresh_schedule(n_steps, refresh)
    sel_want = pm_want = im_want = None
    worst_score = 0.0
    for t in range(n_steps):
        x = gen.next_step()
        q, k, v = (swam.to_device(x[n], wl.dtype) for n in "qkv")
        before = out.clone()
        ctx.step(q, k, v, swam.REFRESH_FULL if sched[t] else swam.REUSE, out)
        ctx.check()
        sc_dev, lse_dev, _ = ctx.cached_scores()
        sel_dev, pm_dev, im_dev = (a.cpu().numpy().copy() for a in ctx.selection())
        dense = sched[t]
        if every_row is not None and t < every_row_steps:
            rows_of = lambda n: all_rows(range(B) if every_row == "all" else [every_row], n)   # noqa: E731
        else:
            rows_of = lambda n: sampled_rows(rng, B, n, H, n_pairs)                             # noqa: E731
        if dense:
            # ---- full step: normalisers, scores (all elements), selection and maps, dense attention rows
            lse64 = ora.action_lse(x["q"], x["k"], H)
            assert np.abs(lse_dev.cpu().numpy() - lse64).max() <= 2e-3, t
            s64 = ora.score(x["q"], x["k"], wl.n_obs, wl.n_frames, wl.n_spatial, H, lse=lse64)
            got_s = sc_dev.cpu().numpy()
            rel = float((np.abs(got_s - s64) / np.maximum(s64, 1e-30)).max())
            worst_score = max(worst_score, rel)
            assert np.abs(got_s - s64).max() <= 1e-4 and rel <= SCORE_REL, (t, rel)
            iso = ora.select(got_s, kc, ks)                       # stage-isolated: the device's own score array
            ipm, iim = ora.maps(iso["sel_idx"], wl.n_obs, wl.n_spatial, H)
            assert np.array_equal(sel_dev, iso["sel_idx"]), t
            assert np.array_equal(pm_dev, ipm) and np.array_equal(im_dev, iim), t
            e2e = ora.select(s64.astype(np.float32), kc, ks)      # end to end: the oracle's scores
            assert np.array_equal(sel_dev, e2e["sel_idx"]), (t, "relative gaps at the three cuts", e2e["margins"],
                                                             "largest relative score error", rel)
            sel_want, pm_want, im_want = sel_dev, pm_dev, im_dev
            rows = rows_of(L)
            want, _ = ora.attention_rows(x["q"], x["k"], x["v"], rows)
            got = out[rows[:, 0], rows[:, 1]].float().cpu().numpy().astype(np.float64)
            check_bf16(got, want, f"step {t} (full)")
        else:
            # ---- sparse step: the selection is the cached one, omitted rows keep their bits, retained rows are the
            # packed attention's
            assert np.array_equal(sel_dev, sel_want) and np.array_equal(pm_dev, pm_want) and np.array_equal(im_dev, im_want), t
            omitted = torch.from_numpy(im_dev < 0).cuda()
            assert int(omitted.sum()) == B * (L - Lp)
            if Lp < L:
                assert torch.equal(out[omitted], before[omitted]), t
            qp, kp, vp = (ora.pack(x[n], pm_dev) for n in "qkv")
            rows = rows_of(Lp)
            want, _ = ora.attention_rows(qp, kp, vp, rows)
            orig = pm_dev[rows[:, 0], rows[:, 1]]
            got = out[rows[:, 0], orig].float().cpu().numpy().astype(np.float64)
            check_bf16(got, want, f"step {t} (sparse)")
        del q, k, v, before
    return worst_score


SCHEDULES = [
    # (workload, every row of the first cycle, every row at every step)
    ("single_view", "all", True),
    ("larger_imagination", "all", False),
    ("multi_view", 5, False),
]


@pytest.mark.parametrize("name,every_row,always", SCHEDULES, ids=[c[0] for c in SCHEDULES])
def test_ten_step_schedule_matches_oracle(name, every_row, always):
    wl = W.WORKLOADS[name]
    assert wl.steps == 10 and wl.refresh == 2
    run_schedule_against_oracle(wl, wl.refresh, wl.steps, every_row, every_row_steps=wl.steps if always else 2)


@pytest.mark.parametrize("keep,refresh", [(0.3, 1), (0.2, 4)], ids=["keep0.3_every_step", "keep0.2_every_4th"])
def test_sweep_shape_refresh_intervals(keep, refresh):
    """App. C.2's other schedules at the sweep shape: a refresh at every step (every step dense: the selection is
    rebuilt each time and never used) and one full step in four."""
    wl = W.sweep_workload(keep, refresh)
    run_schedule_against_oracle(wl, refresh, 10, None, n_pairs=512)
