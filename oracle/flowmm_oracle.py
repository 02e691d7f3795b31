"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, not the product).

Builds `flowmm_oracle.c` with gcc on first use and exposes its steps with
numpy arrays.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may import this module; the CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flowmm_oracle.c")
_BUILD = os.path.join(_HERE, "_build")
_LIB = os.path.join(_BUILD, "libflowmm_oracle.so")
_lib = None


class _Params(ctypes.Structure):
    _fields_ = [
        ("n_units", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("seq_len", ctypes.c_int32), ("window", ctypes.c_int32),
        ("n_keep", ctypes.c_int32),
        ("softmax_scale", ctypes.c_double), ("theta", ctypes.c_double), ("tau", ctypes.c_double),
        ("tau_mode", ctypes.c_int32), ("flow_mode", ctypes.c_int32), ("merge_mode", ctypes.c_int32),
        ("keep_window", ctypes.c_int32),
    ]


TAU_ABS, TAU_REL = 0, 1
FLOW_AUTO, FLOW_FORCE_INTRA, FLOW_FORCE_CROSS, FLOW_MISALIGNED = 0, 1, 2, 3
MERGE_EXPSIM, MERGE_MEAN = 0, 1
INTRA, CROSS = 0, 1


@dataclass
class OracleParams:
    n_units: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_len: int
    window: int
    n_keep: int
    softmax_scale: float = 0.0
    theta: float = 0.25
    tau: float = float("inf")
    tau_mode: int = TAU_ABS
    flow_mode: int = FLOW_AUTO
    merge_mode: int = MERGE_EXPSIM
    keep_window: int = 0

    def c(self) -> _Params:
        return _Params(self.n_units, self.n_q_heads, self.n_kv_heads, self.head_dim, self.seq_len, self.window,
                       self.n_keep, self.softmax_scale, self.theta, self.tau, self.tau_mode, self.flow_mode,
                       self.merge_mode, self.keep_window)


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared library (gcc, -O2, OpenMP)."""
    os.makedirs(_BUILD, exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.flowmm_oracle_cosine.restype = ctypes.c_double
        _lib.flowmm_oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().flowmm_oracle_threads())


def _f32(x):
    return np.ascontiguousarray(x, dtype=np.float32)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def cosine(ki, kj) -> float:
    ki, kj = _f32(ki), _f32(kj)
    return float(_load().flowmm_oracle_cosine(ctypes.c_int32(ki.shape[-1]), _ptr(ki), _ptr(kj)))


def score(p: OracleParams, q, k, modality):
    """-> importance [U,Hkv,L], cross [U,Hq], total [U,Hq] (float64)."""
    q, k = _f32(q), _f32(k)
    m = np.ascontiguousarray(modality, dtype=np.uint8)
    assert q.shape == (p.n_units, p.n_q_heads, p.window, p.head_dim), q.shape
    assert k.shape == (p.n_units, p.n_kv_heads, p.seq_len, p.head_dim), k.shape
    assert m.shape == (p.n_units, p.seq_len), m.shape
    imp = np.zeros((p.n_units, p.n_kv_heads, p.seq_len), dtype=np.float64)
    cross = np.zeros((p.n_units, p.n_q_heads), dtype=np.float64)
    total = np.zeros((p.n_units, p.n_q_heads), dtype=np.float64)
    cp = p.c()
    rc = _load().flowmm_oracle_score(ctypes.byref(cp), _ptr(q), _ptr(k), _ptr(m), _ptr(imp), _ptr(cross), _ptr(total))
    if rc != 0:
        raise ValueError("oracle score: bad shape (code %d)" % rc)
    return imp, cross, total


def layer_flow(p: OracleParams, cross, total):
    """-> rho [U] float64, strategy [U] int32 (1 = cross-modal, 0 = intra-modal)."""
    cross = np.ascontiguousarray(cross, dtype=np.float64)
    total = np.ascontiguousarray(total, dtype=np.float64)
    rho = np.zeros(p.n_units, dtype=np.float64)
    strat = np.zeros(p.n_units, dtype=np.int32)
    cp = p.c()
    _load().flowmm_oracle_layer_flow(ctypes.byref(cp), _ptr(cross), _ptr(total), _ptr(rho), _ptr(strat))
    return rho, strat


def select(p: OracleParams, importance):
    """-> retained [U,Hkv,B], evicted [U,Hkv,L-B], both ascending int32."""
    imp = np.ascontiguousarray(importance, dtype=np.float64)
    assert imp.shape == (p.n_units, p.n_kv_heads, p.seq_len)
    ret = np.zeros((p.n_units, p.n_kv_heads, p.n_keep), dtype=np.int32)
    evi = np.zeros((p.n_units, p.n_kv_heads, p.seq_len - p.n_keep), dtype=np.int32)
    cp = p.c()
    rc = _load().flowmm_oracle_select(ctypes.byref(cp), _ptr(imp), _ptr(ret), _ptr(evi))
    if rc != 0:
        raise ValueError("oracle select: bad budget (code %d)" % rc)
    return ret, evi


def match(p: OracleParams, k, importance, modality, retained, evicted, strategy, row_select=None):
    """-> match [U,Hkv,E] int32, sim [U,Hkv,E], runner_up [U,Hkv,E] float64.  row_select (optional, bool
    [U,Hkv,E]): only these non-pivots are evaluated, the others come back with match = -2."""
    k = _f32(k)
    imp = np.ascontiguousarray(importance, dtype=np.float64)
    m = np.ascontiguousarray(modality, dtype=np.uint8)
    ret = np.ascontiguousarray(retained, dtype=np.int32)
    evi = np.ascontiguousarray(evicted, dtype=np.int32)
    strat = np.ascontiguousarray(strategy, dtype=np.int32)
    E = p.seq_len - p.n_keep
    assert ret.shape == (p.n_units, p.n_kv_heads, p.n_keep) and evi.shape == (p.n_units, p.n_kv_heads, E)
    mt = np.zeros((p.n_units, p.n_kv_heads, E), dtype=np.int32)
    sim = np.zeros((p.n_units, p.n_kv_heads, E), dtype=np.float64)
    ru = np.zeros((p.n_units, p.n_kv_heads, E), dtype=np.float64)
    cp = p.c()
    sel = None
    if row_select is not None:
        sel = np.ascontiguousarray(row_select, dtype=np.uint8)
        assert sel.shape == mt.shape
    _load().flowmm_oracle_match(ctypes.byref(cp), _ptr(k), _ptr(imp), _ptr(m), _ptr(ret), _ptr(evi), _ptr(strat),
                                _ptr(sel) if sel is not None else ctypes.c_void_p(0), _ptr(mt), _ptr(sim), _ptr(ru))
    return mt, sim, ru


def merge(p: OracleParams, k, v, retained, evicted, match_, sim):
    """-> k_out, v_out [U,Hkv,B,D] float64, weight_sum [U,Hkv,B]."""
    k, v = _f32(k), _f32(v)
    ret = np.ascontiguousarray(retained, dtype=np.int32)
    evi = np.ascontiguousarray(evicted, dtype=np.int32)
    mt = np.ascontiguousarray(match_, dtype=np.int32)
    sm = np.ascontiguousarray(sim, dtype=np.float64)
    shape = (p.n_units, p.n_kv_heads, p.n_keep, p.head_dim)
    ko = np.zeros(shape, dtype=np.float64)
    vo = np.zeros(shape, dtype=np.float64)
    z = np.zeros(shape[:3], dtype=np.float64)
    cp = p.c()
    _load().flowmm_oracle_merge(ctypes.byref(cp), _ptr(k), _ptr(v), _ptr(ret), _ptr(evi), _ptr(mt), _ptr(sm),
                                _ptr(ko), _ptr(vo), _ptr(z))
    return ko, vo, z


def compress_layer(p: OracleParams, q, k, v, modality, forced: Optional[Dict[str, np.ndarray]] = None,
                   row_select=None) -> Dict[str, np.ndarray]:
    """The whole path, step by step.  `forced` may replace the decision outputs of a
    step ("importance", "strategy", "retained"+"evicted", "match"+"match_sim") before
    the steps after it run; tests use it to follow a near-tie the other way."""
    forced = forced or {}
    out: Dict[str, np.ndarray] = {}
    imp, cross, total = score(p, q, k, modality)
    out["importance_own"], out["cross"], out["total"] = imp, cross, total
    imp = forced.get("importance", imp)
    out["importance"] = np.asarray(imp, dtype=np.float64)
    rho, strat = layer_flow(p, cross, total)
    out["rho"] = rho
    strat = forced.get("strategy", strat)
    out["strategy"] = np.asarray(strat, dtype=np.int32)
    if "retained" in forced:
        ret, evi = forced["retained"], forced["evicted"]
    else:
        ret, evi = select(p, out["importance"])
    out["retained"], out["evicted"] = np.asarray(ret, dtype=np.int32), np.asarray(evi, dtype=np.int32)
    mt, sim, ru = match(p, k, out["importance"], modality, out["retained"], out["evicted"], out["strategy"], row_select)
    out["match_own"], out["match_sim_own"], out["runner_up"] = mt, sim, ru
    if "match" in forced:
        mt, sim = forced["match"], forced["match_sim"]
    out["match"], out["match_sim"] = np.asarray(mt, dtype=np.int32), np.asarray(sim, dtype=np.float64)
    if row_select is None:
        ko, vo, z = merge(p, k, v, out["retained"], out["evicted"], out["match"], out["match_sim"])
        out["k_out"], out["v_out"], out["weight_sum"] = ko, vo, z
    return out


def decode_attention(q, k, v, scale: float = 0.0) -> np.ndarray:
    """Eq. 4 for one decode step over a cache: q [U,Hq,D], k, v [U,Hkv,N,D] -> out [U,Hq,D] float64."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    U, Hq, D = q.shape
    Hkv, N = k.shape[1], k.shape[2]
    assert k.shape == (U, Hkv, N, D) and v.shape == k.shape
    out = np.zeros((U, Hq, D), dtype=np.float64)
    rc = _load().flowmm_oracle_decode_attention(ctypes.c_int32(U), ctypes.c_int32(Hq), ctypes.c_int32(Hkv),
                                                ctypes.c_int32(D), ctypes.c_int32(N), ctypes.c_double(scale),
                                                _ptr(q), _ptr(k), _ptr(v), _ptr(out))
    if rc != 0:
        raise ValueError("oracle decode_attention: bad shape (code %d)" % rc)
    return out


def recompress(p: OracleParams, q_win, k_cache, v_cache, row_modality) -> Dict[str, np.ndarray]:
    """Re-compression of a cache that has grown during decoding (Eq. 3 appends one row per step; the paper runs
    the compression of Section 3.3 once, after prefill, and does not say what happens afterwards).

    The reading taken: the current cache of a KV head - the rows an earlier compression left, in order, followed by
    the rows appended since - is treated as that head's context of length L' = p.seq_len, and the steps of
    Section 3.3 run on it again with the proxy window taken from the W most recent queries (q_win):
      * a row that came out of an earlier merge is an ordinary token now; its modality is that of the pivot it
        was merged into, which is why modality is given per head and row (row_modality [U, Hkv, L']): after a
        compression the heads of a layer no longer hold the same tokens;
      * importance is taken afresh from the current window (nothing is carried over), the causal mask follows
        the row order (window row a sees cache rows 0 .. L' - W + a), which is the true mask whenever at least W
        rows have been appended;
      * rho stays a property of the layer: the mean over all query heads of the layer (Eq. 6), each head's
        cross-modal mass measured against its own KV head's row modalities; one strategy per unit;
      * merge weights are those of Eq. 5's reading again (a row's earlier merges are not counted).
    Returns the step outputs shaped per (unit, KV head), `row_modality_out` [U, Hkv, B'] for the next round,
    rho [U] and strategy [U].
    """
    U, Hq, Hkv, D, L, W, B = p.n_units, p.n_q_heads, p.n_kv_heads, p.head_dim, p.seq_len, p.window, p.n_keep
    G = Hq // Hkv
    q, k, v = _f32(q_win), _f32(k_cache), _f32(v_cache)
    m = np.ascontiguousarray(row_modality, dtype=np.uint8)
    assert q.shape == (U, Hq, W, D) and k.shape == (U, Hkv, L, D) and v.shape == k.shape and m.shape == (U, Hkv, L)
    # every (unit, KV head) as a problem of its own with one KV head, its G query heads and its own modality map
    ph = OracleParams(U * Hkv, G, 1, D, L, W, B, p.softmax_scale, p.theta, p.tau, p.tau_mode, p.flow_mode,
                      p.merge_mode, p.keep_window)
    qh, kh, vh, mh = q.reshape(U * Hkv, G, W, D), k.reshape(U * Hkv, 1, L, D), v.reshape(U * Hkv, 1, L, D), m.reshape(U * Hkv, L)
    imp, cross, total = score(ph, qh, kh, mh)
    # Eq. 6 over all query heads of the layer
    rho, strat = layer_flow(p, cross.reshape(U, Hq), total.reshape(U, Hq))
    ret, evi = select(ph, imp)
    mt, sim, _ = match(ph, kh, imp, mh, ret, evi, np.repeat(strat, Hkv))
    ko, vo, _ = merge(ph, kh, vh, ret, evi, mt, sim)
    E = L - B
    return {
        "importance": imp.reshape(U, Hkv, L), "cross": cross.reshape(U, Hq), "rho": rho, "strategy": strat,
        "retained": ret.reshape(U, Hkv, B), "evicted": evi.reshape(U, Hkv, E), "match": mt.reshape(U, Hkv, E),
        "match_sim": sim.reshape(U, Hkv, E), "k_out": ko.reshape(U, Hkv, B, D), "v_out": vo.reshape(U, Hkv, B, D),
        "row_modality_out": np.take_along_axis(mh, ret.reshape(U * Hkv, B).astype(np.int64), -1).reshape(U, Hkv, B),
    }
