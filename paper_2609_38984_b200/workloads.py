"""Seeded synthetic workloads shaped like the five benchmark configurations.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only describes shapes and integer budgets
and draws Q/K/V tensors.  The tensors stand in for the activations of a
world-action model (which are not available offline); their structure follows
what the paper observes about action-to-future attention (Sec. 3.2): each
future frame is attended by its own contiguous group of action queries, the
attended region is a spatial hotspot that differs between frames, and the
hotspot barely moves between consecutive denoising steps.

Sequence order is [observed | future frame 0 .. F-1 | action]; tensors are
[B, L, N_h, D], token-major.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Tuple

import numpy as np

F32 = 0
BF16 = 1


def budgets_from_keep(keep: float, n_spatial: int) -> Tuple[int, int]:
    """Integer per-frame budgets (K_c, K_s) for a keep ratio.

    The paper only gives integer budgets (Table 5: 80 core + 104 anchors of 360)
    and defines the pruning ratio as r = 1 - K/N_s (Sec. 5.4).  The rule used for
    the benchmark shapes is K = round-half-up(keep * N_s) and a 10:13 split
    (80:104) between core tokens and shared anchors.
    """
    k = int(math.floor(keep * n_spatial + 0.5))
    k = max(0, min(k, n_spatial))
    k_core = int(math.floor(k * 10.0 / 23.0 + 0.5))
    return k_core, k - k_core


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_obs: int
    n_frames: int
    views: int
    grid_h: int
    grid_w: int
    n_action: int
    n_heads: int
    head_dim: int
    dtype: int
    keep: float
    steps: int
    refresh: int
    seed: int
    blobs: int = 0          # hotspots per (view, frame); 0 = plain i.i.d. N(0,1)
    rho: float = 0.8        # AR(1) coefficient of future/action tensors across steps
    blob_logit: float = 4.0  # logit added at a hotspot centre
    blob_sigma: float = 3.0  # hotspot width in patches
    k_core: Optional[int] = None
    k_anchor: Optional[int] = None
    n_kv_heads: Optional[int] = None   # key/value heads (grouped-query attention); None = n_heads

    @property
    def kv_heads(self) -> int:
        return self.n_heads if self.n_kv_heads is None else self.n_kv_heads

    @property
    def n_spatial(self) -> int:
        return self.views * self.grid_h * self.grid_w

    @property
    def budgets(self) -> Tuple[int, int]:
        if self.k_core is not None and self.k_anchor is not None:
            return self.k_core, self.k_anchor
        return budgets_from_keep(self.keep, self.n_spatial)

    @property
    def k_keep(self) -> int:
        return sum(self.budgets)

    @property
    def seq_len(self) -> int:
        return self.n_obs + self.n_frames * self.n_spatial + self.n_action

    @property
    def packed_len(self) -> int:
        return self.n_obs + self.n_frames * self.k_keep + self.n_action

    @property
    def group(self) -> int:
        return self.n_action // self.n_frames

    @property
    def row_elems(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == F32 else 2

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    # batch 1; 2 x 8x8 future tokens, 16 observed, 8 action; 2 heads x 32; fp32; i.i.d. N(0,1)
    "tiny": Workload("tiny", 1, 16, 2, 1, 8, 8, 8, 2, 32, F32, 0.5, 3, 2, 0, blobs=0),
    # 4 x 24x24 future, 576 observed, 32 action; 24 x 64; bf16
    "single_view": Workload("single_view", 1, 576, 4, 1, 24, 24, 32, 24, 64, BF16, 0.25, 10, 2, 1, blobs=1),
    # 8 x 32x32 future, 1024 observed, 64 action; 32 x 128; bf16; two hotspots per frame
    "larger_imagination": Workload("larger_imagination", 1, 1024, 8, 1, 32, 32, 64, 32, 128, BF16, 0.3, 10, 2, 2, blobs=2),
    # batch 8, 3 views x 4 x 24x24 future, 1728 observed, 32 action; 24 x 64; bf16
    "multi_view": Workload("multi_view", 8, 1728, 4, 3, 24, 24, 32, 24, 64, BF16, 0.25, 10, 2, 3, blobs=1),
}

# Shapes of the models the paper evaluates (Table 5 and App. B.2): camera views, future latent frames, tokens per
# future frame, denoising steps, the integer budgets K_c + K_s, and the action horizon of 32 tokens that all three
# backbones share, which gives four frame-aligned queries per future frame for the Cosmos models (8 frames) and
# sixteen for FastWAM-Joint (2 frames).  refresh = steps means that only the first step is a full step, the paper's
# default (Sec. 4.2).  The paper does not print head counts, head sizes or the size of the observed frame: those are
# stand-ins (one observed latent frame of N_s tokens).  Cosmos 3 Edge's three views differ in size (340 tokens per
# frame do not split into three equal grids), so it is laid out as one 20 x 17 grid.
PAPER_ACTION_HORIZON = 32
PAPER_SHAPES: Dict[str, Workload] = {
    "cosmos3_nano": Workload("cosmos3_nano", 1, 360, 8, 3, 10, 12, PAPER_ACTION_HORIZON, 16, 128, BF16, 184 / 360, 4, 4, 11,
                             blobs=1, k_core=80, k_anchor=104),
    "cosmos3_edge": Workload("cosmos3_edge", 1, 340, 8, 1, 20, 17, PAPER_ACTION_HORIZON, 16, 128, BF16, 184 / 340, 4, 4, 12,
                             blobs=2, k_core=80, k_anchor=104),
    "fastwam_joint": Workload("fastwam_joint", 1, 98, 2, 2, 7, 7, PAPER_ACTION_HORIZON, 12, 64, BF16, 31 / 98, 10, 10, 13,
                              blobs=1, k_core=19, k_anchor=12),
}

# Retained tokens per frame in the paper's pruning-ratio ablation on 360-token frames (Sec. 5.4: ratios 28.89 %,
# 48.89 % (the default 184) and 68.89 %)
PAPER_PRUNING_BUDGETS = (256, 184, 112)

# Selection strategies of the component ablation (Sec. 5.4), all at the same K per frame
SELECT_VARIANTS = ("combined", "core_only", "stable_only", "random")


def variant_workload(wl: Workload, variant: str, k_keep: Optional[int] = None) -> Workload:
    """The workload with the budgets of a selection variant: `combined` keeps the workload's own split (or the 10:13
    rule for a new K), `core_only` spends all K on frame-specific core tokens, `stable_only` all K on shared anchors,
    `random` ranks caller-drawn random keys per frame, which is core_only on those keys."""
    if variant not in SELECT_VARIANTS:
        raise ValueError(f"unknown selection variant {variant!r}")
    k = wl.k_keep if k_keep is None else int(k_keep)
    if not 0 <= k <= wl.n_spatial:
        raise ValueError("K must lie in [0, N_s]")
    if variant == "combined":
        if k_keep is None:
            kc, ks = wl.budgets
        else:
            kc = int(math.floor(k * 10.0 / 23.0 + 0.5))
            ks = k - kc
    elif variant == "stable_only":
        kc, ks = 0, k
    else:
        kc, ks = k, 0
    return wl.with_(name=f"{wl.name}_{variant}_k{k}", k_core=kc, k_anchor=ks, keep=k / wl.n_spatial)


SWEEP_KEEPS = (0.1, 0.2, 0.3, 0.5, 1.0)
SWEEP_REFRESH = (1, 2, 4)


def sweep_workload(keep: float, refresh: int) -> Workload:
    """The keep-ratio x refresh-interval sweep runs at the larger-imagination shape with seed 4."""
    base = WORKLOADS["larger_imagination"]
    return base.with_(name=f"sweep_keep{keep:g}_r{refresh}", keep=keep, refresh=refresh, seed=4)


def refresh_schedule(steps: int, refresh: int) -> List[bool]:
    """True where a denoising step is a full (refresh) step: every `refresh`-th step from step 0."""
    return [(t % refresh) == 0 for t in range(steps)]


# ----------------------------------------------------------------------------
# bf16 helpers (storage only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round to nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# generator
# ----------------------------------------------------------------------------
_TENSOR_ID = {"q": 0, "k": 1, "v": 2}
_CHUNK_ROWS = 512


def _normal_rows(seed: int, step: int, tensor: int, b: int, n_rows: int, row_elems: int, stream: int) -> np.ndarray:
    """[n_rows, row_elems] float32 N(0,1), reproducible per (seed, step, tensor, sample, stream), drawn in
    parallel chunks with one counter-based generator key per chunk."""
    out = np.empty((n_rows, row_elems), dtype=np.float32)
    n_chunks = (n_rows + _CHUNK_ROWS - 1) // _CHUNK_ROWS

    def fill(c: int) -> None:
        lo = c * _CHUNK_ROWS
        hi = min(n_rows, lo + _CHUNK_ROWS)
        key = [(seed << 40) | (step << 20) | (tensor << 8) | stream, (b << 32) | c]
        g = np.random.Generator(np.random.Philox(key=key))
        out[lo:hi] = g.standard_normal((hi - lo, row_elems), dtype=np.float32)

    if n_chunks == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(fill, range(n_chunks)))
    return out


class Generator:
    """Draws the Q/K/V tensors of one workload step by step.

    Observed-token rows are fixed across steps.  Future and action rows follow
    x_t = rho * x_{t-1} + sqrt(1 - rho^2) * n_t (tiny: rho = 0, fresh noise each
    step).  When the workload has hotspots, each (sample, view, frame) carries
    `blobs` Gaussian bumps whose centres start uniform on the patch grid and move
    by at most one patch per axis per step; along a seeded unit direction
    u[f, h] the future keys of frame f get amplitude a * bump(j) and the action
    queries of the frame's query group get amplitude a, with a^2 / sqrt(D) =
    blob_logit, so a hotspot centre raises the aligned logit by `blob_logit`.
    """

    def __init__(self, wl: Workload):
        self.wl = wl
        self._t = -1
        self._base: Dict[str, np.ndarray] = {}
        rng = np.random.Generator(np.random.Philox(key=[wl.seed, 0xB10B]))
        if wl.blobs > 0:
            self._centres = rng.uniform(
                0.0, 1.0, size=(wl.batch, wl.views, wl.n_frames, wl.blobs, 2)
            ) * np.array([wl.grid_h - 1, wl.grid_w - 1], dtype=np.float64)
            u = rng.standard_normal((wl.n_frames, wl.n_heads, wl.head_dim))
            self._u = (u / np.linalg.norm(u, axis=-1, keepdims=True)).astype(np.float32)
        else:
            self._centres = None
            self._u = None
        self._drift_rng = np.random.Generator(np.random.Philox(key=[wl.seed, 0xD21F7]))

    # -- hotspot geometry -------------------------------------------------
    def centres(self) -> Optional[np.ndarray]:
        return None if self._centres is None else self._centres.copy()

    def _bump(self) -> np.ndarray:
        """[B, F, N_s] float32: sum of Gaussian bumps, within-frame order view-major."""
        wl = self.wl
        yy, xx = np.meshgrid(np.arange(wl.grid_h), np.arange(wl.grid_w), indexing="ij")
        pos = np.stack([yy.reshape(-1), xx.reshape(-1)], axis=-1).astype(np.float64)  # [hw, 2]
        c = self._centres  # [B, views, F, blobs, 2]
        d2 = ((pos[None, None, None, None, :, :] - c[:, :, :, :, None, :]) ** 2).sum(-1)  # [B,views,F,blobs,hw]
        g = np.exp(-d2 / (2.0 * wl.blob_sigma ** 2)).sum(axis=3)  # [B, views, F, hw]
        g = np.transpose(g, (0, 2, 1, 3)).reshape(wl.batch, wl.n_frames, wl.n_spatial)
        return g.astype(np.float32)

    # -- stepping ---------------------------------------------------------
    def next_step(self) -> Dict[str, np.ndarray]:
        """Advance one denoising step; returns float32 arrays q [B, L, N_h, D] and k, v [B, L, N_kv, D] whose values
        are already rounded to the workload's storage type (bf16 workloads: bf16-representable)."""
        wl = self.wl
        self._t += 1
        t = self._t
        rho = wl.rho if wl.blobs > 0 else 0.0
        n_fut = wl.n_frames * wl.n_spatial
        out: Dict[str, np.ndarray] = {}
        if t > 0 and self._centres is not None:
            drift = self._drift_rng.uniform(-1.0, 1.0, size=self._centres.shape)
            hi = np.array([wl.grid_h - 1, wl.grid_w - 1], dtype=np.float64)
            self._centres = np.clip(self._centres + drift, 0.0, hi)
        bump = self._bump() if self._centres is not None else None
        amp = math.sqrt(wl.blob_logit * math.sqrt(wl.head_dim))
        for name, tid in _TENSOR_ID.items():
            if t == 0:
                base = np.empty((wl.batch, wl.seq_len, wl.row_elems), dtype=np.float32)
                for b in range(wl.batch):
                    base[b] = _normal_rows(wl.seed, 0, tid, b, wl.seq_len, wl.row_elems, 0)
                self._base[name] = base
            else:
                base = self._base[name]
                c1 = np.float32(math.sqrt(1.0 - rho * rho))
                for b in range(wl.batch):
                    noise = _normal_rows(wl.seed, t, tid, b, wl.seq_len - wl.n_obs, wl.row_elems, 1)
                    dyn = base[b, wl.n_obs:]
                    dyn *= np.float32(rho)
                    noise *= c1
                    dyn += noise
            x = base.reshape(wl.batch, wl.seq_len, wl.n_heads, wl.head_dim).copy()
            if bump is not None and name == "k":
                fut = x[:, wl.n_obs:wl.n_obs + n_fut].reshape(
                    wl.batch, wl.n_frames, wl.n_spatial, wl.n_heads, wl.head_dim)
                fut += np.float32(amp) * bump[:, :, :, None, None] * self._u[None, :, None, :, :]
            grp = wl.n_heads // wl.kv_heads
            if bump is not None and name == "q":
                act = x[:, wl.n_obs + n_fut:].reshape(
                    wl.batch, wl.n_frames, wl.group, wl.n_heads, wl.head_dim)
                # every query head points along the direction of the key head it reads
                u_q = self._u if grp == 1 else np.repeat(self._u[:, ::grp], grp, axis=1)
                act += np.float32(amp) * u_q[None, :, None, :, :]
            if grp > 1 and name in ("k", "v"):
                x = np.ascontiguousarray(x[:, :, ::grp])      # grouped-query attention: one K/V head per group
            if wl.dtype == BF16:
                x = bf16_bits_to_f32(f32_to_bf16_bits(x)).reshape(x.shape)
            out[name] = x
        return out


def generate_steps(wl: Workload, n_steps: Optional[int] = None) -> List[Dict[str, np.ndarray]]:
    g = Generator(wl)
    return [g.next_step() for _ in range(wl.steps if n_steps is None else n_steps)]


def random_scores(seed: int, batch: int, n_frames: int, n_spatial: int, ties: bool = False) -> np.ndarray:
    """[B, F, N_s] float32 positive score arrays for testing selection alone; `ties` quantises them so
    that many exact ties occur."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x5C0]))
    s = rng.gamma(0.7, 1.0, size=(batch, n_frames, n_spatial)).astype(np.float32) / np.float32(n_spatial)
    if ties:
        s = (np.floor(s * np.float32(n_spatial * 4)) / np.float32(n_spatial * 4)).astype(np.float32)
    return s
