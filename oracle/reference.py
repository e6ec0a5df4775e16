"""CPU oracle of the sparse denoising step: Python front end of swam_oracle.c.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the product path.  It shares no code
with the CUDA library.  Arithmetic is fp64 (numpy / the C file); scores are
stored as float32 before selection, which is the one precision the method's
ranking is defined in here (both sides rank the same stored type).

Parity unpinned: the approximation quality of the sparse output against the
dense one (the paper reports task success only); it is reported, not asserted.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swam_oracle.c")
_LIB = os.path.join(_HERE, "libswam_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, OpenMP, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: Optional[np.ndarray], t):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(t))


def threads() -> int:
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


# ----------------------------------------------------------------------------
# stage definitions
# ----------------------------------------------------------------------------
def query_weights(g: int) -> np.ndarray:
    """alpha within one frame-aligned query group: the central half of the group weighs twice the outer
    quarters, normalised to sum to one (App. B.2: (1,2,2,1)/6 for groups of four)."""
    if g % 4 != 0:
        raise ValueError("the 2:1 rule needs a group size divisible by 4")
    w = np.ones(g, dtype=np.float64)
    w[g // 4: g - g // 4] = 2.0
    return w / w.sum()


def expand_kv(x: np.ndarray, n_heads: int) -> np.ndarray:
    """Grouped-query attention written out: a key/value tensor with fewer heads than the queries is the tensor in
    which query head h finds key/value head h // (N_h / N_kv); repeating each head N_h / N_kv times gives the plain
    multi-head problem every function below is defined on."""
    n_kv = x.shape[2]
    if n_kv == n_heads:
        return x
    assert n_heads % n_kv == 0, "the number of query heads must be a multiple of the key/value heads"
    return np.repeat(x, n_heads // n_kv, axis=2)


SEES_OBSERVED, SEES_FUTURE, SEES_ALL = 0, 1, 2


def key_limits(rows: np.ndarray, obs_end: int, fut_end: int, n: int, sees: Sequence[int]) -> np.ndarray:
    """Visible-key count of each listed (b, r) row under segment-prefix visibility: the sequence is
    [observed | future | action] with the observed tokens ending at obs_end and the future tokens at fut_end; a row of
    segment s sees the keys up to the end of the segment sees[s] names (observed, future, or everything)."""
    ends = np.array([obs_end, fut_end, n], dtype=np.int32)
    r = np.asarray(rows).reshape(-1, 2)[:, 1]
    seg = (r >= obs_end).astype(np.int32) + (r >= fut_end).astype(np.int32)
    return ends[np.asarray(sees, dtype=np.int32)[seg]].astype(np.int32)


def attention_rows(q: np.ndarray, k: np.ndarray, v: np.ndarray, rows: np.ndarray,
                   scale: Optional[float] = None, key_limit: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Softmax attention (Sec. 3.1) for the listed (b, r) query rows, all heads.
    q: [B, n, N_h, D], k, v: [B, n, N_h or N_kv, D] float32.  key_limit: per listed row, the number of leading keys it
    sees (None = all).  Returns out [n_rows, N_h, D], lse [n_rows, N_h] (float64)."""
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(expand_kv(k, q.shape[2]), dtype=np.float32)
    v = np.ascontiguousarray(expand_kv(v, q.shape[2]), dtype=np.float32)
    _, n, nh, d = q.shape
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 2)
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    out = np.empty((rows.shape[0], nh, d), dtype=np.float64)
    lse = np.empty((rows.shape[0], nh), dtype=np.float64)
    lib.oracle_attention_rows(_p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float),
                              ctypes.c_int(n), ctypes.c_int(nh), ctypes.c_int(d), ctypes.c_double(scale),
                              _p(rows, ctypes.c_int32), ctypes.c_int64(rows.shape[0]),
                              _p(out, ctypes.c_double), _p(lse, ctypes.c_double),
                              None if key_limit is None else _p(np.ascontiguousarray(key_limit, dtype=np.int32), ctypes.c_int32))
    return out, lse


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: Optional[float] = None,
              visibility: Optional[Tuple[int, int, Sequence[int]]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """All rows: out [B, n, N_h, D], lse [B, N_h, n].  visibility = (obs_end, fut_end, sees) restricts each row to
    the key prefix its segment sees (see key_limits); None = every row sees every key."""
    b, n, nh, d = q.shape
    rows = np.stack(np.meshgrid(np.arange(b), np.arange(n), indexing="ij"), axis=-1).reshape(-1, 2)
    lim = None if visibility is None else key_limits(rows, visibility[0], visibility[1], n, visibility[2])
    out, lse = attention_rows(q, k, v, rows, scale, lim)
    return out.reshape(b, n, nh, d), np.ascontiguousarray(lse.reshape(b, n, nh).transpose(0, 2, 1))


def action_lse(q: np.ndarray, k: np.ndarray, n_action: int, scale: Optional[float] = None,
               n_visible: Optional[int] = None) -> np.ndarray:
    """lambda_h(i): log-sum-exp of the action queries over the keys they see: all keys of the full sequence, or its
    first n_visible keys (App. A.2: "over all visible keys").  [B, N_h, H]."""
    b, n, nh, d = q.shape
    rows = np.stack(np.meshgrid(np.arange(b), np.arange(n - n_action, n), indexing="ij"), axis=-1).reshape(-1, 2)
    lim = None if n_visible is None else np.full(rows.shape[0], n_visible, dtype=np.int32)
    _, lse = attention_rows(q, k, np.zeros_like(k, dtype=np.float32), rows, scale, lim)
    return np.ascontiguousarray(lse.reshape(b, n_action, nh).transpose(0, 2, 1))


def score(q: np.ndarray, k: np.ndarray, n_obs: int, n_frames: int, n_spatial: int, n_action: int,
          lse: Optional[np.ndarray] = None, alpha: Optional[np.ndarray] = None,
          scale: Optional[float] = None) -> np.ndarray:
    """Spatial score S [B, F, N_s] (Eq. 12), float64."""
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(expand_kv(k, q.shape[2]), dtype=np.float32)
    b, n, nh, d = q.shape
    assert n == n_obs + n_frames * n_spatial + n_action and n_action % n_frames == 0
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    if lse is None:
        lse = action_lse(q, k, n_action, scale)
    lse = np.ascontiguousarray(lse, dtype=np.float64)
    alpha = query_weights(n_action // n_frames) if alpha is None else np.ascontiguousarray(alpha, dtype=np.float64)
    s = np.empty((b, n_frames, n_spatial), dtype=np.float64)
    lib.oracle_score(_p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(lse, ctypes.c_double),
                     _p(alpha, ctypes.c_double), ctypes.c_int(b), ctypes.c_int(n_obs), ctypes.c_int(n_frames),
                     ctypes.c_int(n_spatial), ctypes.c_int(n_action), ctypes.c_int(nh), ctypes.c_int(d),
                     ctypes.c_double(scale), _p(s, ctypes.c_double))
    return s


def quality(scores_f32: np.ndarray) -> np.ndarray:
    """(R, E, Q) of Eq. 9 per sample from the stored scores [B, F, N_s]; returns [B, 3] float64."""
    lib = _load()
    s = np.ascontiguousarray(scores_f32, dtype=np.float32)
    out = np.empty((s.shape[0], 3), dtype=np.float64)
    for b in range(s.shape[0]):
        lib.oracle_quality(_p(s[b], ctypes.c_float), ctypes.c_int(s.shape[1]), ctypes.c_int(s.shape[2]),
                           _p(out[b], ctypes.c_double))
    return out


def select(scores_f32: np.ndarray, k_core: int, k_anchor: int, beta: float = 1.0) -> Dict[str, np.ndarray]:
    """Pool / core / anchor selection (Eq. 4-6, 10-11) per sample on stored float32 scores [B, F, N_s].
    Returns sel_idx [B, F, K] ascending plus the intermediate sets and the TopK cut margins."""
    lib = _load()
    s = np.ascontiguousarray(scores_f32, dtype=np.float32)
    assert s.dtype == np.float32
    b, f, n = s.shape
    k = k_core + k_anchor
    res = dict(sel_idx=np.zeros((b, f, k), np.int32), pool=np.zeros((b, n), np.uint8),
               core=np.zeros((b, f, n), np.uint8), anchors=np.zeros((b, k_anchor), np.int32),
               anchor_key=np.zeros((b, n), np.float64), margins=np.zeros((b, 3), np.float64))
    for i in range(b):
        lib.oracle_select(_p(s[i], ctypes.c_float), ctypes.c_int(f), ctypes.c_int(n), ctypes.c_int(k_core),
                          ctypes.c_int(k_anchor), ctypes.c_double(beta), _p(res["sel_idx"][i], ctypes.c_int32),
                          _p(res["pool"][i], ctypes.c_uint8), _p(res["core"][i], ctypes.c_uint8),
                          _p(res["anchors"][i], ctypes.c_int32), _p(res["anchor_key"][i], ctypes.c_double),
                          _p(res["margins"][i], ctypes.c_double))
    return res


def aggregate(layer_scores: np.ndarray, layer_quality: np.ndarray, k_layer: int):
    """Multi-layer aggregation (Eq. 3, Eq. 11): layer_scores [n_layers, B, F, N_s] float32, layer_quality
    [n_layers, B, 3] float32 (R, E, Q per layer, Eq. 9).  Returns v_core, v_all [B, F, N_s] float32 and the chosen
    core layers [B, k_layer] (ascending)."""
    lib = _load()
    ls = np.ascontiguousarray(layer_scores, dtype=np.float32)
    nl, b, f, n = ls.shape
    lq = np.ascontiguousarray(layer_quality, dtype=np.float32)
    v_core = np.empty((b, f, n), np.float32)
    v_all = np.empty((b, f, n), np.float32)
    layers = np.empty((b, min(k_layer, nl)), np.int32)
    for i in range(b):
        si = np.ascontiguousarray(ls[:, i].reshape(nl, f * n))
        qi = np.ascontiguousarray(lq[:, i, 2])
        lib.oracle_aggregate(_p(si, ctypes.c_float), _p(qi, ctypes.c_float), ctypes.c_int(nl), ctypes.c_int(k_layer),
                             ctypes.c_int(f * n), _p(v_core[i], ctypes.c_float), _p(v_all[i], ctypes.c_float),
                             _p(layers[i], ctypes.c_int32))
    return v_core, v_all, layers


def select2(v_core: np.ndarray, v_all: np.ndarray, k_core: int, k_anchor: int, beta: float = 1.0) -> np.ndarray:
    """Selection with the core score map V for pool and cores and V_all for the anchors; sel_idx [B, F, K]."""
    lib = _load()
    vc = np.ascontiguousarray(v_core, dtype=np.float32)
    va = np.ascontiguousarray(v_all, dtype=np.float32)
    b, f, n = vc.shape
    sel = np.zeros((b, f, k_core + k_anchor), np.int32)
    for i in range(b):
        lib.oracle_select2(_p(vc[i], ctypes.c_float), _p(va[i], ctypes.c_float), ctypes.c_int(f), ctypes.c_int(n),
                           ctypes.c_int(k_core), ctypes.c_int(k_anchor), ctypes.c_double(beta), _p(sel[i], ctypes.c_int32))
    return sel


def maps(sel_idx: np.ndarray, n_obs: int, n_spatial: int, n_action: int) -> Tuple[np.ndarray, np.ndarray]:
    """pack_map [B, L'] and inv_map [B, L] (Sec. 4.2 packing metadata)."""
    lib = _load()
    sel = np.ascontiguousarray(sel_idx, dtype=np.int32)
    b, f, k = sel.shape
    L = n_obs + f * n_spatial + n_action
    Lp = n_obs + f * k + n_action
    pack = np.empty((b, Lp), np.int32)
    inv = np.empty((b, L), np.int32)
    for i in range(b):
        lib.oracle_maps(_p(sel[i], ctypes.c_int32), ctypes.c_int(n_obs), ctypes.c_int(f), ctypes.c_int(n_spatial),
                        ctypes.c_int(n_action), ctypes.c_int(k), _p(pack[i], ctypes.c_int32),
                        _p(inv[i], ctypes.c_int32))
    return pack, inv


def pack(x: np.ndarray, pack_map: np.ndarray) -> np.ndarray:
    """Xp[b, p] = X[b, pack_map[b, p]]."""
    return np.stack([x[b][pack_map[b]] for b in range(x.shape[0])])


def scatter(out_p: np.ndarray, pack_map: np.ndarray, cached: np.ndarray) -> np.ndarray:
    """Eq. 7: current values on retained rows, cached values elsewhere."""
    out = cached.copy()
    for b in range(out.shape[0]):
        out[b][pack_map[b]] = out_p[b]
    return out


def overlap(p: np.ndarray, q: np.ndarray) -> float:
    """Eq. 13 on two non-negative arrays, each normalised to sum to one."""
    p = np.asarray(p, np.float64).reshape(-1)
    q = np.asarray(q, np.float64).reshape(-1)
    return float(np.minimum(p / p.sum(), q / q.sum()).sum())


# ----------------------------------------------------------------------------
# the step loop (Sec. 4.2): full steps build the selection and fill the cache,
# sparse steps reuse both
# ----------------------------------------------------------------------------
class StepState:
    def __init__(self):
        self.out: Optional[np.ndarray] = None      # [B, L, N_h, D] float64, persistent across steps
        self.scores: Optional[np.ndarray] = None   # float32 [B, F, N_s]
        self.sel: Optional[Dict[str, np.ndarray]] = None
        self.pack_map: Optional[np.ndarray] = None
        self.inv_map: Optional[np.ndarray] = None
        self.sees: Optional[Sequence[int]] = None    # segment-prefix visibility of the backbone, None = full
        self.n_obs = 0
        self.n_action = 0


def full_step(st: StepState, q, k, v, n_obs, n_frames, n_spatial, n_action, k_core, k_anchor,
              beta: float = 1.0, rows: Optional[np.ndarray] = None, scale: Optional[float] = None,
              sees: Optional[Sequence[int]] = None) -> StepState:
    """Dense joint attention over all L tokens, then score, select and build the maps.
    With `rows` given only those (b, r) rows of the dense output are computed (sampled parity at full size);
    st.out then holds NaN elsewhere.  sees: segment-prefix visibility (see key_limits), None = full."""
    b, n, nh, d = q.shape
    obs_end, fut_end = n_obs, n_obs + n_frames * n_spatial
    vis = None if sees is None else (obs_end, fut_end, sees)
    st.sees, st.n_obs, st.n_action = sees, n_obs, n_action
    if rows is None:
        out, lse = attention(q, k, v, scale, vis)
        lse_act = np.ascontiguousarray(lse[:, :, n - n_action:])
        st.out = out
    else:
        lim = None if sees is None else key_limits(rows, obs_end, fut_end, n, sees)
        o, _ = attention_rows(q, k, v, rows, scale, lim)
        st.out = np.full((b, n, nh, d), np.nan)
        st.out[rows[:, 0], rows[:, 1]] = o
        lse_act = action_lse(q, k, n_action, scale, None if sees is None else [obs_end, fut_end, n][sees[2]])
    s64 = score(q, k, n_obs, n_frames, n_spatial, n_action, lse=lse_act, scale=scale)
    st.scores = s64.astype(np.float32)
    st.sel = select(st.scores, k_core, k_anchor, beta)
    st.pack_map, st.inv_map = maps(st.sel["sel_idx"], n_obs, n_spatial, n_action)
    return st


def _packed_visibility(st: "StepState", n_p: int):
    """(obs_end, fut_end, sees) of the packed sequence [observed | F * K retained | action], or None."""
    if st.sees is None:
        return None
    return (st.n_obs, n_p - st.n_action, st.sees)


def sparse_step(st: StepState, q, k, v, rows_packed: Optional[np.ndarray] = None,
                scale: Optional[float] = None) -> np.ndarray:
    """Pack by the cached map, attend over the compact sequence, scatter back (Eq. 7).  Returns the packed
    attention output ([B, L', N_h, D], or the listed packed rows when `rows_packed` is given)."""
    assert st.pack_map is not None, "a full step must come first"
    qp, kp, vp = pack(q, st.pack_map), pack(k, st.pack_map), pack(v, st.pack_map)
    n_p = qp.shape[1]
    if rows_packed is None:
        op, _ = attention(qp, kp, vp, scale, _packed_visibility(st, n_p))
        st.out = scatter(op, st.pack_map, st.out)
        return op
    vis = _packed_visibility(st, n_p)
    lim = None if vis is None else key_limits(rows_packed, vis[0], vis[1], n_p, vis[2])
    o, _ = attention_rows(qp, kp, vp, rows_packed, scale, lim)
    orig = st.pack_map[rows_packed[:, 0], rows_packed[:, 1]]
    st.out[rows_packed[:, 0], orig] = o
    return o


def run_steps(steps: Sequence[Dict[str, np.ndarray]], refresh: int, n_obs, n_frames, n_spatial, n_action,
              k_core, k_anchor, beta: float = 1.0, sees: Optional[Sequence[int]] = None) -> List[Dict[str, np.ndarray]]:
    """All denoising steps of one action chunk; step t is a full step when t % refresh == 0."""
    st = StepState()
    log = []
    for t, x in enumerate(steps):
        is_full = (t % refresh) == 0
        if is_full:
            full_step(st, x["q"], x["k"], x["v"], n_obs, n_frames, n_spatial, n_action, k_core, k_anchor, beta, sees=sees)
        else:
            sparse_step(st, x["q"], x["k"], x["v"])
        log.append(dict(full=is_full, out=st.out.copy(), scores=st.scores.copy(),
                        sel_idx=st.sel["sel_idx"].copy(), pack_map=st.pack_map.copy(),
                        inv_map=st.inv_map.copy(), margins=st.sel["margins"].copy()))
    return log
