"""Tracing: every launching call of the library opens an NVTX range named after itself in the domain "swam", and a step
opens one range per stage inside its own.  The tests attach a tiny NVTX tool (tests/nvtx_probe.c, loaded by the NVTX
loader through NVTX_INJECTION64_PATH) in a child process and read the ranges it recorded."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_2609_38984_b200 import build as swam_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def probe(tmp_path_factory):
    swam_build.build_library()
    so = str(tmp_path_factory.mktemp("nvtx") / "nvtx_probe.so")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    subprocess.check_call(["gcc", "-shared", "-fPIC", "-O1", f"-I{cuda}/include", "-o", so,
                           os.path.join(ROOT, "tests", "nvtx_probe.c")])
    return so


def traced(probe, tmp_path, code):
    """Runs `code` in a child process with the probe attached; returns the recorded lines."""
    log = str(tmp_path / "ranges.txt")
    env = dict(os.environ, NVTX_INJECTION64_PATH=probe, SWAM_NVTX_PROBE_OUT=log, PYTHONPATH=ROOT)
    subprocess.run([sys.executable, "-c", textwrap.dedent(code)], env=env, cwd=ROOT, check=True, timeout=600)
    return open(log).read().split("\n")[:-1] if os.path.exists(log) else []


def tree(lines):
    """Nested (name, children) lists from the push/pop lines of the domain; fails on unbalanced ranges."""
    root = ("", [])
    stack = [root]
    for ln in lines:
        if ln.startswith("push "):
            node = (ln[5:], [])
            stack[-1][1].append(node)
            stack.append(node)
        elif ln == "pop":
            assert len(stack) > 1, "pop without a push"
            stack.pop()
    assert len(stack) == 1, "a range was left open"
    return root[1]


def test_calls_open_and_close_their_range_even_when_they_fail(probe, tmp_path):
    lines = traced(probe, tmp_path, """
        import ctypes
        from paper_2609_38984_b200 import swam
        lib = swam.load_library()
        assert lib.swam_step(None, None, None, None, 0, None, None) == swam.ERR_INVALID_ARG
        assert lib.swam_select(None, None, None, None, None, None) == swam.ERR_INVALID_ARG
        assert lib.swam_check(None, None) != 0
    """)
    assert lines[0] == "domain swam"
    assert [n for n, kids in tree(lines)] == ["swam_step", "swam_select", "swam_check"]
    assert all(not kids for _, kids in tree(lines))


@pytest.mark.gpu
def test_a_refresh_cycle_shows_its_stages_as_nested_ranges(probe, tmp_path):
    lines = traced(probe, tmp_path, """
        from paper_2609_38984_b200 import swam, workloads as W
        wl = W.WORKLOADS["single_view"]
        x = W.Generator(wl).next_step()
        q, k, v = (swam.to_device(x[n], wl.dtype) for n in "qkv")
        ctx = swam.Swam.from_workload(wl)
        out = ctx.empty_full().zero_()
        ctx.step(q, k, v, swam.REFRESH_FULL, out)
        ctx.step(q, k, v, swam.REUSE, out)
        ctx.set_option(swam.OPT_SPARSE_PATH, swam.SPARSE_STAGED)
        ctx.step(q, k, v, swam.REFRESH_LIGHT, out)
        ctx.check()
    """)
    steps = [(n, [c[0] for c in kids]) for n, kids in tree(lines) if n == "swam_step"]
    assert steps == [
        ("swam_step", ["dense_attention", "swam_score", "select"]),
        ("swam_step", ["swam_pack", "packed_attention"]),
        ("swam_step", ["swam_score", "select", "swam_pack", "packed_attention", "swam_scatter"]),
    ]
    assert tree(lines)[-1][0] == "swam_check"
