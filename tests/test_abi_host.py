"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects bad shapes
before touching the device."""
import numpy as np
import ctypes
import os
import re

import pytest

from paper_2609_38984_b200 import build as swam_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    swam_build.build_library()
    from paper_2609_38984_b200 import swam
    return swam.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "swam.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(swam_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2609_38984_b200 import swam
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(swam.EXPORTS) == names
    assert b"sm_100a" in lib.swam_version()


def _create(lib, **kw):
    from paper_2609_38984_b200 import swam
    base = dict(batch=1, n_obs=16, n_frames=2, n_spatial=64, n_action=8, n_heads=2, head_dim=32, k_core=14,
                k_anchor=18, dtype=0, softmax_scale=0.0, cv_beta=1.0, n_kv_heads=0)
    base.update(kw)
    weights = base.pop("weights", None)
    arr = (ctypes.c_float * len(weights))(*weights) if weights else None
    base["query_weights"] = ctypes.cast(arr, ctypes.POINTER(ctypes.c_float)) if arr else None
    sh = swam.SwamShape(*[base[f] for f, _ in swam.SwamShape._fields_])
    ctx = ctypes.c_void_p()
    rc = lib.swam_create(ctypes.byref(sh), ctypes.byref(ctx))
    if rc == 0:
        lib.swam_destroy(ctx)
    return rc


def test_shape_validation_happens_on_the_host(lib):
    from paper_2609_38984_b200 import swam
    assert _create(lib, n_action=7) == swam.ERR_INVALID_ARG               # H not divisible by F
    assert _create(lib, k_core=40, k_anchor=30) == swam.ERR_INVALID_ARG   # K_c + K_s > N_s
    assert _create(lib, n_action=12) == swam.ERR_INVALID_ARG              # group of 6 without explicit weights
    assert _create(lib, head_dim=48) == swam.ERR_UNSUPPORTED
    assert _create(lib, dtype=3) == swam.ERR_INVALID_ARG
    assert _create(lib, batch=0) == swam.ERR_INVALID_ARG
    assert _create(lib, n_action=12, weights=[0.5] * 6) == swam.ERR_INVALID_ARG   # weights must sum to one
    assert _create(lib, n_action=128) == swam.ERR_UNSUPPORTED             # group of 64 exceeds the scorer's limit
    assert _create(lib, n_heads=6, n_kv_heads=4) == swam.ERR_INVALID_ARG  # key/value heads must divide the heads
    assert _create(lib, n_heads=6, n_kv_heads=-1) == swam.ERR_INVALID_ARG
    assert _create(lib, n_heads=6, n_kv_heads=2) in (0, swam.ERR_CUDA)   # a valid shape; no device on a CPU-only host
    assert lib.swam_create(None, None) == swam.ERR_INVALID_ARG


def test_null_context_calls_fail_cleanly(lib):
    from paper_2609_38984_b200 import swam
    n = ctypes.c_size_t()
    assert lib.swam_workspace_bytes(None, ctypes.byref(n)) == swam.ERR_INVALID_ARG
    assert lib.swam_step(None, None, None, None, 0, None, None) == swam.ERR_INVALID_ARG
    assert lib.swam_check(None, None) == swam.ERR_INVALID_ARG
    assert lib.swam_last_error(None) == b"null context"


def test_shapes_beyond_the_selection_kernels_shared_memory_are_rejected(lib):
    from paper_2609_38984_b200 import swam
    # F * N_s scores (two maps) + keys + flags must fit one SM's shared memory
    assert _create(lib, n_frames=8, n_spatial=8192, n_action=32, k_core=10, k_anchor=10) == swam.ERR_UNSUPPORTED
    assert _create(lib, n_obs=1 << 25) == swam.ERR_UNSUPPORTED            # sequence length limit
    assert _create(lib, batch=70000, n_obs=0, n_frames=1, n_spatial=64, n_action=4, k_core=8, k_anchor=8) == swam.ERR_UNSUPPORTED   # samples are a grid dimension


def test_degree4_exp2_polynomial_bound():
    """The softmax pass of the head-dim-64 attention kernel evaluates one exponential in eight as
    2^round(x) * p(x - round(x)); this pins the coefficients' error bound against the library exp2."""
    c = [0.9999992847442627, 0.6931217908859253, 0.240247443318367, 0.05591785907745361, 0.009570102207362652]
    f = np.linspace(-0.5, 0.5, 200001)
    p = ((((c[4] * f + c[3]) * f + c[2]) * f + c[1]) * f + c[0])
    assert np.abs(p / np.exp2(f) - 1).max() < 3e-6
