"""Thin Python binding of libswam.so (argument marshalling only).

Every step of the path runs in the library's CUDA kernels; torch is used here
for device memory and streams.  There is no CPU fallback: if the shared
library is missing or cannot be loaded, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import workloads as W

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libswam.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_STATE, ERR_CUDA, ERR_DEVICE_CHECK, ERR_TIMEOUT = range(8)
F32, BF16 = 0, 1
REUSE, REFRESH_FULL, REFRESH_LIGHT = 0, 1, 2
OPT_ATTN_VARIANT, OPT_SPARSE_PATH, OPT_VISIBILITY, OPT_HOST_ROWS = 1, 2, 3, 4
HOST_ROWS_RETAINED, HOST_ROWS_ALL = 0, 1
SEES_OBSERVED, SEES_FUTURE, SEES_ALL = 0, 1, 2
ATTN_AUTO, ATTN_WARP_MMA = 0, 1
SPARSE_FUSED, SPARSE_STAGED, SPARSE_FUSED_KV = 0, 1, 2

EXPORTS = [
    "swam_create", "swam_destroy", "swam_workspace_bytes", "swam_bind_workspace", "swam_score", "swam_score_noalloc",
    "swam_select", "swam_aggregate", "swam_select_maps",
    "swam_pack", "swam_sparse_attn", "swam_scatter", "swam_step", "swam_host_io_bytes", "swam_bind_host_io",
    "swam_step_host", "swam_host_join", "swam_get_selection", "swam_get_scores", "swam_set_selection", "swam_state_bytes",
    "swam_state_export", "swam_state_import", "swam_check", "swam_selftest_timeout", "swam_launch_floor", "swam_set_option", "swam_launch_count",
    "swam_last_error", "swam_version",
]


class SwamShape(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_obs", ctypes.c_int32), ("n_frames", ctypes.c_int32),
        ("n_spatial", ctypes.c_int32), ("n_action", ctypes.c_int32), ("n_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("k_core", ctypes.c_int32), ("k_anchor", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("cv_beta", ctypes.c_float),
        ("query_weights", ctypes.POINTER(ctypes.c_float)), ("n_kv_heads", ctypes.c_int32),
    ]


class SwamError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"swam error {code}: {msg}")
        self.code = code


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libswam.so; raises if it has not been built (python -m paper_2609_38984_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_38984_b200.build`; "
                               "there is no CPU fallback")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        lib.swam_create.argtypes = [ctypes.POINTER(SwamShape), ctypes.POINTER(vp)]
        lib.swam_destroy.argtypes = [vp]
        lib.swam_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
        lib.swam_bind_workspace.argtypes = [vp, vp, ctypes.c_size_t]
        lib.swam_host_io_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
        lib.swam_bind_host_io.argtypes = [vp, vp, ctypes.c_size_t]
        lib.swam_score.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        lib.swam_score_noalloc.argtypes = [vp, vp, vp, vp, vp]
        lib.swam_select.argtypes = [vp, vp, vp, vp, vp, vp]
        lib.swam_aggregate.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp]
        lib.swam_select_maps.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        lib.swam_pack.argtypes = [vp] * 9
        lib.swam_sparse_attn.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp]
        lib.swam_scatter.argtypes = [vp] * 7
        lib.swam_step.argtypes = [vp, vp, vp, vp, i32, vp, vp]
        lib.swam_step_host.argtypes = [vp, vp, vp, vp, i32, vp, vp]
        lib.swam_host_join.argtypes = [vp, vp]
        lib.swam_get_selection.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp)]
        lib.swam_get_scores.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp)]
        lib.swam_set_selection.argtypes = [vp, vp, vp, vp, vp]
        lib.swam_state_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
        lib.swam_state_export.argtypes = [vp, vp, vp]
        lib.swam_state_import.argtypes = [vp, vp, vp]
        lib.swam_check.argtypes = [vp, vp]
        lib.swam_selftest_timeout.argtypes = [vp, ctypes.c_uint64, vp]
        lib.swam_launch_floor.argtypes = [vp, vp]
        lib.swam_set_option.argtypes = [vp, i32, i32]
        lib.swam_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_int64)]
        lib.swam_last_error.argtypes = [vp]
        lib.swam_last_error.restype = ctypes.c_char_p
        lib.swam_version.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def torch_dtype(dtype: int) -> torch.dtype:
    return torch.float32 if dtype == F32 else torch.bfloat16


class Swam:
    """One context = one shape.  Methods mirror the C entry points and take CUDA tensors laid out
    [B, L, N_h, D] (or [B, L', N_h, D] for packed tensors); K and V have n_kv_heads heads instead of N_h."""

    def __init__(self, batch, n_obs, n_frames, n_spatial, n_action, n_heads, head_dim, k_core, k_anchor,
                 dtype=BF16, softmax_scale: float = 0.0, cv_beta: float = 1.0, query_weights=None,
                 device: Optional[torch.device] = None, bind: bool = True, n_kv_heads: int = 0):
        self.lib = load_library()
        self._weights = None
        if query_weights is not None:
            self._weights = (ctypes.c_float * len(query_weights))(*[float(x) for x in query_weights])
        self.shape = SwamShape(batch, n_obs, n_frames, n_spatial, n_action, n_heads, head_dim, k_core, k_anchor,
                               dtype, softmax_scale, cv_beta,
                               ctypes.cast(self._weights, ctypes.POINTER(ctypes.c_float)) if self._weights else None,
                               n_kv_heads)
        self.ctx = ctypes.c_void_p()
        if device is None:
            if not torch.cuda.is_available():
                raise RuntimeError("swam needs a CUDA device; there is no CPU fallback")
            device = torch.device("cuda", torch.cuda.current_device())
        self.device = device
        rc = self.lib.swam_create(ctypes.byref(self.shape), ctypes.byref(self.ctx))
        if rc != OK:
            self.ctx = ctypes.c_void_p()
            raise SwamError(rc, "swam_create rejected the shape")
        self.B, self.F, self.N_s, self.H = batch, n_frames, n_spatial, n_action
        self.n_obs, self.N_h, self.D = n_obs, n_heads, head_dim
        self.N_kv = n_kv_heads if n_kv_heads > 0 else n_heads
        self.K = k_core + k_anchor
        self.L = n_obs + n_frames * n_spatial + n_action
        self.Lp = n_obs + n_frames * self.K + n_action
        self.dtype = dtype
        self.workspace = None
        self.staging = None
        if bind:
            self.bind_workspace()

    @classmethod
    def from_workload(cls, wl: W.Workload, **kw) -> "Swam":
        kc, ks = wl.budgets
        return cls(wl.batch, wl.n_obs, wl.n_frames, wl.n_spatial, wl.n_action, wl.n_heads, wl.head_dim, kc, ks,
                   dtype=wl.dtype, n_kv_heads=wl.kv_heads, **kw)

    def __del__(self):
        try:
            if getattr(self, "ctx", None) and self.ctx.value:
                self.lib.swam_destroy(self.ctx)
                self.ctx = ctypes.c_void_p()
        except Exception:
            pass

    # -- helpers -----------------------------------------------------------
    def _chk(self, rc: int):
        if rc != OK:
            raise SwamError(rc, self.lib.swam_last_error(self.ctx).decode())

    def workspace_bytes(self) -> int:
        n = ctypes.c_size_t()
        self._chk(self.lib.swam_workspace_bytes(self.ctx, ctypes.byref(n)))
        return n.value

    def bind_workspace(self):
        self.workspace = torch.empty(self.workspace_bytes() + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._chk(self.lib.swam_bind_workspace(self.ctx, ctypes.c_void_p(self.workspace.data_ptr() + off),
                                               self.workspace.numel() - off))

    def host_io_bytes(self) -> int:
        n = ctypes.c_size_t()
        self._chk(self.lib.swam_host_io_bytes(self.ctx, ctypes.byref(n)))
        return n.value

    def bind_host_io(self):
        self.staging = torch.empty(self.host_io_bytes() + 256, dtype=torch.uint8, device=self.device)
        off = (-self.staging.data_ptr()) % 256
        self._chk(self.lib.swam_bind_host_io(self.ctx, ctypes.c_void_p(self.staging.data_ptr() + off),
                                             self.staging.numel() - off))

    def empty_full(self) -> torch.Tensor:
        return torch.empty((self.B, self.L, self.N_h, self.D), dtype=torch_dtype(self.dtype), device=self.device)

    def empty_packed(self, kv: bool = False) -> torch.Tensor:
        return torch.empty((self.B, self.Lp, self.N_kv if kv else self.N_h, self.D), dtype=torch_dtype(self.dtype),
                           device=self.device)

    # -- the calls ---------------------------------------------------------
    def score(self, q, k, lse_action=None, quality: bool = False):
        scores = torch.empty((self.B, self.F, self.N_s), dtype=torch.float32, device=self.device)
        qual = torch.empty((self.B, 3), dtype=torch.float32, device=self.device) if quality else None
        self._chk(self.lib.swam_score(self.ctx, _ptr(q), _ptr(k), _ptr(lse_action), _ptr(scores), _ptr(qual), _stream()))
        return (scores, qual) if quality else scores

    def score_noalloc(self, q, k, scores):
        """Scores into the caller's `scores` tensor using the library's built-in scratch: no workspace, nothing
        allocated (for callers that cannot obtain device memory at call time)."""
        self._chk(self.lib.swam_score_noalloc(self.ctx, _ptr(q), _ptr(k), _ptr(scores), _stream()))
        return scores

    def select(self, scores) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        sel = torch.empty((self.B, self.F, self.K), dtype=torch.int32, device=self.device)
        pack = torch.empty((self.B, self.Lp), dtype=torch.int32, device=self.device)
        inv = torch.empty((self.B, self.L), dtype=torch.int32, device=self.device)
        self._chk(self.lib.swam_select(self.ctx, _ptr(scores), _ptr(sel), _ptr(pack), _ptr(inv), _stream()))
        return sel, pack, inv

    def aggregate(self, layer_scores, layer_quality, k_layer: int):
        """V, V_all and the chosen core layers from per-layer scores [n_layers, B, F, N_s] and qualities [n_layers, B, 3]."""
        n_layers = layer_scores.shape[0]
        v_core = torch.empty((self.B, self.F, self.N_s), dtype=torch.float32, device=self.device)
        v_all = torch.empty_like(v_core)
        layers = torch.empty((self.B, k_layer), dtype=torch.int32, device=self.device)
        self._chk(self.lib.swam_aggregate(self.ctx, _ptr(layer_scores), _ptr(layer_quality), n_layers, k_layer,
                                          _ptr(v_core), _ptr(v_all), _ptr(layers), _stream()))
        return v_core, v_all, layers

    def select_maps(self, core_scores, anchor_scores):
        sel = torch.empty((self.B, self.F, self.K), dtype=torch.int32, device=self.device)
        pack = torch.empty((self.B, self.Lp), dtype=torch.int32, device=self.device)
        inv = torch.empty((self.B, self.L), dtype=torch.int32, device=self.device)
        self._chk(self.lib.swam_select_maps(self.ctx, _ptr(core_scores), _ptr(anchor_scores), _ptr(sel), _ptr(pack),
                                            _ptr(inv), _stream()))
        return sel, pack, inv

    def pack(self, q, k, v, pack_map):
        outs = [self.empty_packed(kv=i > 0) if x is not None else None for i, x in enumerate((q, k, v))]
        self._chk(self.lib.swam_pack(self.ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(pack_map), _ptr(outs[0]),
                                     _ptr(outs[1]), _ptr(outs[2]), _stream()))
        return outs

    def sparse_attn(self, qp, kp, vp, want_lse: bool = False):
        n = qp.shape[1]
        out = torch.empty_like(qp)
        lse = torch.empty((self.B, self.N_h, n), dtype=torch.float32, device=self.device) if want_lse else None
        self._chk(self.lib.swam_sparse_attn(self.ctx, _ptr(qp), _ptr(kp), _ptr(vp), n, _ptr(out), _ptr(lse), _stream()))
        return (out, lse) if want_lse else out

    def scatter(self, out_p, pack_map, inv_map, cached, out=None):
        out = cached if out is None else out
        self._chk(self.lib.swam_scatter(self.ctx, _ptr(out_p), _ptr(pack_map), _ptr(inv_map), _ptr(cached), _ptr(out),
                                        _stream()))
        return out

    def step(self, q, k, v, mode: int, out):
        self._chk(self.lib.swam_step(self.ctx, _ptr(q), _ptr(k), _ptr(v), mode, _ptr(out), _stream()))
        return out

    def step_host(self, q_host, k_host, v_host, mode: int, out_host):
        """Host (pinned) tensors in and out; copies and kernels are enqueued on the current stream."""
        if self.staging is None:
            self.bind_host_io()
        self._chk(self.lib.swam_step_host(self.ctx, _ptr(q_host), _ptr(k_host), _ptr(v_host), mode, _ptr(out_host),
                                          _stream()))
        return out_host

    def host_join(self):
        """The current stream waits for the last step_host result to arrive in its host buffer."""
        self._chk(self.lib.swam_host_join(self.ctx, _stream()))

    def _view(self, ptr: ctypes.c_void_p, shape, dtype) -> torch.Tensor:
        off = ptr.value - self.workspace.data_ptr()
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        return self.workspace[off:off + nbytes].view(dtype).view(*shape)

    def selection(self):
        """Views of the cached sel_idx, pack_map, inv_map inside the workspace."""
        a, b, c = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p()
        self._chk(self.lib.swam_get_selection(self.ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
        return (self._view(a, (self.B, self.F, self.K), torch.int32), self._view(b, (self.B, self.Lp), torch.int32),
                self._view(c, (self.B, self.L), torch.int32))

    def set_selection(self, sel_idx: torch.Tensor, pack_map: torch.Tensor, inv_map: torch.Tensor):
        """Install a selection made elsewhere (another context's, or swam_select on other scores) for REUSE steps."""
        for t, shape in ((sel_idx, (self.B, self.F, self.K)), (pack_map, (self.B, self.Lp)), (inv_map, (self.B, self.L))):
            if t.dtype != torch.int32 or tuple(t.shape) != shape or not t.is_contiguous() or not t.is_cuda:
                raise ValueError(f"expected a contiguous int32 CUDA tensor of shape {shape}")
        self._chk(self.lib.swam_set_selection(self.ctx, _ptr(sel_idx), _ptr(pack_map), _ptr(inv_map), _stream()))

    def export_state(self) -> torch.Tensor:
        """The cross-step state (scores, diagnostics, normalisers, selection, maps) as one opaque byte tensor."""
        n = ctypes.c_size_t()
        self._chk(self.lib.swam_state_bytes(self.ctx, ctypes.byref(n)))
        buf = torch.empty(n.value, dtype=torch.uint8, device=self.device)
        self._chk(self.lib.swam_state_export(self.ctx, _ptr(buf), _stream()))
        return buf

    def import_state(self, buf: torch.Tensor):
        n = ctypes.c_size_t()
        self._chk(self.lib.swam_state_bytes(self.ctx, ctypes.byref(n)))
        if buf.dtype != torch.uint8 or buf.numel() != n.value or not buf.is_cuda or not buf.is_contiguous():
            raise ValueError(f"expected a contiguous uint8 CUDA tensor of {n.value} bytes")
        self._chk(self.lib.swam_state_import(self.ctx, _ptr(buf), _stream()))

    def cached_scores(self):
        a, b, c = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p()
        self._chk(self.lib.swam_get_scores(self.ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
        return (self._view(a, (self.B, self.F, self.N_s), torch.float32),
                self._view(b, (self.B, self.N_h, self.H), torch.float32), self._view(c, (self.B, 3), torch.float32))

    def check(self):
        self._chk(self.lib.swam_check(self.ctx, _stream()))

    def selftest_timeout(self, limit_cycles: int = 100_000):
        """Enqueue the wait self-test: the next check() raises SwamError(ERR_TIMEOUT)."""
        self._chk(self.lib.swam_selftest_timeout(self.ctx, limit_cycles, _stream()))

    def set_option(self, option: int, value: int):
        self._chk(self.lib.swam_set_option(self.ctx, option, value))

    def set_visibility(self, observed_rows_see: int, future_rows_see: int, action_rows_see: int):
        """Segment-prefix visibility: what the rows of each segment see (SEES_OBSERVED / SEES_FUTURE / SEES_ALL)."""
        self.set_option(OPT_VISIBILITY, observed_rows_see | (future_rows_see << 2) | (action_rows_see << 4))

    def launch_count(self) -> int:
        n = ctypes.c_int64()
        self._chk(self.lib.swam_launch_count(self.ctx, ctypes.byref(n)))
        return n.value


def to_device(x, dtype: int, device=None) -> torch.Tensor:
    """numpy float32 [B, L, N_h, D] (already storage-exact) -> CUDA tensor of the workload dtype."""
    t = torch.from_numpy(x)
    return t.to(device or "cuda", dtype=torch_dtype(dtype)).contiguous()
