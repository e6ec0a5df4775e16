"""The allocation-free scoring entry point against the regular one.

Some callers of the library cannot obtain device memory when they need scores: a serving process whose framework
took all of the GPU's memory at start-up, or a control-loop thread for which cudaMalloc's device-wide stall is not
acceptable.  swam_score_noalloc serves them from scratch that is built into the library; this test checks that it
returns what swam_score returns, on two calls in a row with different inputs (the second call finds the first
call's leftovers in the shared scratch).  The file name keeps it last in collection order.
"""
import numpy as np
import pytest
import torch

from paper_2609_38984_b200 import workloads as W

pytestmark = pytest.mark.gpu

SCORE_REL = 1e-5


@pytest.mark.parametrize("name,kw", [
    ("single_view", dict(n_obs=70, grid_h=10, grid_w=9, n_heads=3)),
    ("tiny", dict()),
], ids=["bf16", "f32"])
def test_noalloc_scores_match_regular_entry_point_twice(name, kw):
    from paper_2609_38984_b200 import swam
    wl = W.WORKLOADS[name].with_(**kw)
    steps = W.generate_steps(wl, 2)
    regular = swam.Swam.from_workload(wl)                 # has a workspace
    bare = swam.Swam.from_workload(wl, bind=False)        # no workspace at all
    for x in steps:
        q, k = swam.to_device(x["q"], wl.dtype), swam.to_device(x["k"], wl.dtype)
        want = regular.score(q, k)                        # normalisers computed in workspace scratch
        got = torch.full_like(want, float("nan"))
        bare.score_noalloc(q, k, got)
        torch.cuda.synchronize()
        w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.abs(g - w).max() <= 1e-4
        assert (np.abs(g - w) / np.maximum(w, 1e-30)).max() <= SCORE_REL


def test_noalloc_rejects_shapes_beyond_the_built_in_scratch():
    from paper_2609_38984_b200 import swam
    big = swam.Swam(64, 4096, 8, 1024, 128, 32, 128, 10, 10, dtype=swam.BF16, bind=False)
    t = torch.zeros(16, device="cuda")
    with pytest.raises(swam.SwamError) as e:
        big.score_noalloc(t, t, t)
    assert e.value.code == swam.ERR_UNSUPPORTED and "scratch" in str(e.value)
