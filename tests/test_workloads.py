"""Host-side checks of the synthetic workload generator (no GPU)."""
import os

import numpy as np

from paper_2609_38984_b200 import workloads as W


def test_shapes_of_the_benchmark_configurations():
    want = {  # name: (L, L', K, row bytes)
        "tiny": (152, 88, 32, 256),
        "single_view": (2912, 1184, 144, 3072),
        "larger_imagination": (9280, 3544, 307, 8192),
        "multi_view": (8672, 3488, 432, 3072),
    }
    for name, (L, Lp, K, row) in want.items():
        wl = W.WORKLOADS[name]
        assert (wl.seq_len, wl.packed_len, wl.k_keep, wl.row_elems * wl.elem_bytes) == (L, Lp, K, row)
        assert wl.n_action % wl.n_frames == 0 and wl.group % 4 == 0
    assert W.sweep_workload(1.0, 4).packed_len == 9280


def test_generator_is_deterministic_and_storage_exact():
    wl = W.WORKLOADS["single_view"].with_(n_obs=40, grid_h=6, grid_w=6, n_heads=2, head_dim=16)
    a = W.generate_steps(wl, 3)
    b = W.generate_steps(wl, 3)
    for x, y in zip(a, b):
        for name in "qkv":
            assert np.array_equal(x[name], y[name])
            assert x[name].shape == (wl.batch, wl.seq_len, wl.n_heads, wl.head_dim)
            # values are exactly representable in bf16
            assert np.array_equal(W.bf16_bits_to_f32(W.f32_to_bf16_bits(x[name])).reshape(x[name].shape), x[name])
    # observed rows are fixed across steps, the rest evolves
    assert np.array_equal(a[0]["k"][:, :wl.n_obs], a[2]["k"][:, :wl.n_obs])
    assert not np.array_equal(a[0]["k"][:, wl.n_obs:], a[1]["k"][:, wl.n_obs:])


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 3.1415927], np.float32)
    bits = W.f32_to_bf16_bits(x)
    back = W.bf16_bits_to_f32(bits)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.0 + 2.0 ** -6 and back[3] == -2.5
    assert abs(back[4] - 3.140625) < 1e-7


def test_hotspot_drift_is_bounded():
    wl = W.WORKLOADS["single_view"].with_(n_obs=8, grid_h=8, grid_w=8, n_heads=1, head_dim=16)
    g = W.Generator(wl)
    g.next_step()
    c0 = g.centres()
    g.next_step()
    c1 = g.centres()
    assert np.abs(c1 - c0).max() <= 1.0 and c1.min() >= 0 and c1.max() <= 7


def test_refresh_schedule():
    assert W.refresh_schedule(5, 2) == [True, False, True, False, True]
    assert W.refresh_schedule(3, 1) == [True, True, True]


def test_paper_shapes_and_ablation_budgets():
    """Table 5: tokens per future frame, future frames, denoising steps and K_c + K_s of the evaluated models."""
    want = {"cosmos3_nano": (360, 8, 4, 80, 104), "cosmos3_edge": (340, 8, 4, 80, 104), "fastwam_joint": (98, 2, 10, 19, 12)}
    for name, (n_s, frames, steps, kc, ks) in want.items():
        wl = W.PAPER_SHAPES[name]
        assert (wl.n_spatial, wl.n_frames, wl.steps, wl.budgets) == (n_s, frames, steps, (kc, ks))
        assert wl.n_action % wl.n_frames == 0 and wl.group % 4 == 0
        # the default schedule: only the first step is a full step
        assert W.refresh_schedule(wl.steps, wl.refresh) == [True] + [False] * (wl.steps - 1)
    # App. B.2: action horizon and aligned queries per frame, as stored in the golden file
    golden = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "budgets.txt")
    rows = [ln.split() for ln in open(golden) if ln.startswith("queries ")]
    assert len(rows) == 3
    for _, name, horizon, per_frame in rows:
        wl = W.PAPER_SHAPES[name]
        assert (wl.n_action, wl.group) == (int(horizon), int(per_frame))
    nano = W.PAPER_SHAPES["cosmos3_nano"]
    # pruning ratios of the ablation: 1 - K / N_s
    assert [round(100 * (1 - k / nano.n_spatial), 2) for k in W.PAPER_PRUNING_BUDGETS] == [28.89, 48.89, 68.89]
    assert W.variant_workload(nano, "combined").budgets == (80, 104)
    assert W.variant_workload(nano, "core_only").budgets == (184, 0)
    assert W.variant_workload(nano, "stable_only").budgets == (0, 184)
    assert W.variant_workload(nano, "random").budgets == (184, 0)
    for k in W.PAPER_PRUNING_BUDGETS:
        kc, ks = W.variant_workload(nano, "combined", k).budgets
        assert kc + ks == k and abs(kc / k - 10 / 23) < 0.01
        assert W.variant_workload(nano, "combined", k).packed_len == nano.n_obs + nano.n_frames * k + nano.n_action
