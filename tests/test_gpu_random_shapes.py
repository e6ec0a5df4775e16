"""Seeded random shapes (head dim, frames, query group, frame size, observed length, heads, grouped heads, batch, keep
ratio) through the paths that depend on them most: the one-pass scorer against the oracle on every element; a
full / reuse / light-refresh schedule with the fused sparse step against the staged one (bit for bit; with 128 or more
observed tokens the fused step reads whole key tiles of them from the full tensors); and the same schedule through the
host-buffer entry point against the device one (bit for bit; the reuse step brings only its retained rows across)."""
import numpy as np
import pytest
import torch

from oracle import reference as ora
from paper_2609_38984_b200 import workloads as W

pytestmark = pytest.mark.gpu

N_CASES = 24


def random_workload(case):
    rng = np.random.default_rng(9000 + case)
    D = int(rng.choice([64, 128]))
    F = int(rng.choice([1, 2, 3, 4, 6, 8]))
    g = int(rng.choice([4, 8, 16]))
    n_heads = int(rng.choice([1, 2, 3, 4]))
    n_kv = int(rng.choice([d for d in (1, 2, 4) if n_heads % d == 0]))
    base = "larger_imagination" if D == 128 else "single_view"
    return W.WORKLOADS[base].with_(
        batch=int(rng.choice([1, 2, 3])), n_obs=int(rng.choice([0, 8, 70, 128, 131, 200, 256, 300, 384, 520, 1024])),
        n_frames=F, views=1, grid_h=int(rng.integers(3, 33)), grid_w=int(rng.integers(3, 33)), n_action=F * g,
        n_heads=n_heads, n_kv_heads=n_kv, keep=float(rng.choice([0.1, 0.25, 0.5, 0.8, 1.0])), steps=3, seed=9000 + case)


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_shape(case):
    from paper_2609_38984_b200 import swam
    wl = random_workload(case)
    steps = W.generate_steps(wl, 3)
    modes = [swam.REFRESH_FULL, swam.REUSE, swam.REFRESH_LIGHT]

    x = steps[0]
    ctx = swam.Swam.from_workload(wl)
    k64 = ora.expand_kv(x["k"], wl.n_heads)
    lse64 = ora.action_lse(x["q"], k64, wl.n_action)
    want = ora.score(x["q"], k64, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, lse=lse64)
    got = ctx.score(swam.to_device(x["q"], wl.dtype), swam.to_device(x["k"], wl.dtype)).cpu().numpy().astype(np.float64)
    ctx.check()
    rel = (np.abs(got - want) / np.maximum(want, 1e-30)).max()
    assert np.isfinite(got).all() and rel <= 1e-5, (wl, rel)

    outs = {}
    for path in (swam.SPARSE_FUSED, swam.SPARSE_STAGED):
        c = swam.Swam.from_workload(wl)
        c.set_option(swam.OPT_SPARSE_PATH, path)
        out = c.empty_full().zero_()
        outs[path] = []
        for xx, mode in zip(steps, modes):
            c.step(*(swam.to_device(xx[n], wl.dtype) for n in "qkv"), mode, out)
            c.check()
            outs[path].append(out.clone())
    for t in range(3):
        assert torch.equal(outs[swam.SPARSE_FUSED][t], outs[swam.SPARSE_STAGED][t]), (wl, t)

    ch = swam.Swam.from_workload(wl)
    tdt = outs[swam.SPARSE_FUSED][0].dtype
    host_in = [[torch.from_numpy(xx[n]).to(tdt).pin_memory() for n in "qkv"] for xx in steps]
    host_out = [torch.empty(outs[swam.SPARSE_FUSED][0].shape, dtype=tdt).pin_memory() for _ in steps]
    for t in range(3):
        ch.step_host(*host_in[t], modes[t], host_out[t])
    ch.check()
    for t in range(3):
        assert torch.equal(outs[swam.SPARSE_FUSED][t].cpu(), host_out[t]), (wl, t)
