"""Python binding of the C ABI in include/flowmm.h.

Argument marshalling only: every function here has the name of the C entry
point it calls, takes torch CUDA tensors where the C function takes device
pointers, and does no arithmetic of its own.  There is no fallback: if
libflowmm.so is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import math
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libflowmm.so")

F32, BF16 = 0, 1
INTRA, CROSS = 0, 1
MERGE_EXPSIM, MERGE_MEAN = 0, 1
TAU_ABS, TAU_REL = 0, 1
FLOW_AUTO, FLOW_FORCE_INTRA, FLOW_FORCE_CROSS, FLOW_MISALIGNED = 0, 1, 2, 3
PATH_AUTO, PATH_SIMT = 0, 1

EXPORTS = (
    "flowmm_workspace_bytes", "flowmm_score", "flowmm_layer_flow", "flowmm_select", "flowmm_match", "flowmm_merge",
    "flowmm_compress_layer", "flowmm_last_device_status", "flowmm_last_launch_count", "flowmm_status_string",
    "flowmm_profile_enable", "flowmm_profile_read", "flowmm_merge_static", "flowmm_selftest_wait_timeout",
    "flowmm_decode_workspace_bytes", "flowmm_decode_attention",
    "flowmm_full_flow_workspace_bytes", "flowmm_full_flow",
    "flowmm_merge_static_status", "flowmm_merge_static_poke_status",
    "flowmm_recompress_workspace_bytes", "flowmm_recompress", "flowmm_debug_build",
)


class FlowmmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (status %d)" % (where, status_string(code), code))


class _CParams(ctypes.Structure):
    _fields_ = [
        ("n_units", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("seq_len", ctypes.c_int32), ("window", ctypes.c_int32),
        ("n_keep", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("theta", ctypes.c_float), ("tau", ctypes.c_float),
        ("tau_mode", ctypes.c_int32), ("flow_mode", ctypes.c_int32), ("merge_mode", ctypes.c_int32),
        ("keep_window", ctypes.c_int32), ("path", ctypes.c_int32),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3), ("v_stride", ctypes.c_int64 * 3),
        ("ko_stride", ctypes.c_int64 * 3), ("vo_stride", ctypes.c_int64 * 3),
    ]


@dataclass
class Params:
    """Mirror of flowmm_params; strides default to dense tensors and are refreshed from the
    tensors each call receives."""
    n_units: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_len: int
    window: int
    n_keep: int
    dtype: int = BF16
    softmax_scale: float = 0.0
    theta: float = 0.25
    tau: float = math.inf
    tau_mode: int = TAU_ABS
    flow_mode: int = FLOW_AUTO
    merge_mode: int = MERGE_EXPSIM
    keep_window: int = 0
    path: int = PATH_AUTO

    @property
    def n_evict(self) -> int:
        return self.seq_len - self.n_keep

    def _dense(self, heads, tokens):
        D = self.head_dim
        return (heads * tokens * D, tokens * D, D)

    def c(self, q=None, k=None, v=None, ko=None, vo=None) -> _CParams:
        def strides(t, heads, tokens):
            if t is None:
                return self._dense(heads, tokens)
            if t.dim() != 4 or t.stride(3) != 1:
                raise ValueError("expected a [units, heads, tokens, head_dim] tensor with contiguous head_dim")
            return (t.stride(0), t.stride(1), t.stride(2))
        cp = _CParams(self.n_units, self.n_q_heads, self.n_kv_heads, self.head_dim, self.seq_len, self.window,
                      self.n_keep, self.dtype, self.softmax_scale, self.theta, self.tau, self.tau_mode,
                      self.flow_mode, self.merge_mode, self.keep_window, self.path)
        cp.q_stride = (ctypes.c_int64 * 3)(*strides(q, self.n_q_heads, self.window))
        cp.k_stride = (ctypes.c_int64 * 3)(*strides(k, self.n_kv_heads, self.seq_len))
        cp.v_stride = (ctypes.c_int64 * 3)(*strides(v, self.n_kv_heads, self.seq_len))
        cp.ko_stride = (ctypes.c_int64 * 3)(*strides(ko, self.n_kv_heads, self.n_keep))
        cp.vo_stride = (ctypes.c_int64 * 3)(*strides(vo, self.n_kv_heads, self.n_keep))
        return cp


_lib = None


def load() -> ctypes.CDLL:
    """Load libflowmm.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                "%s is missing: build it with `python -m paper_2511_05534_b200.build` "
                "(there is no fallback implementation)" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(lib, name)
        lib.flowmm_status_string.restype = ctypes.c_char_p
        lib.flowmm_last_launch_count.restype = ctypes.c_int32
        lib.flowmm_profile_enable.restype = ctypes.c_int
        lib.flowmm_profile_read.restype = ctypes.c_int32
        for name in EXPORTS[:8]:
            getattr(lib, name).restype = ctypes.c_int
        lib.flowmm_merge_static.restype = ctypes.c_int
        lib.flowmm_merge_static_status.restype = ctypes.c_int
        lib.flowmm_recompress_workspace_bytes.restype = ctypes.c_int
        lib.flowmm_recompress.restype = ctypes.c_int
        lib.flowmm_debug_build.restype = ctypes.c_int32
        lib.flowmm_merge_static_poke_status.restype = ctypes.c_int
        lib.flowmm_selftest_wait_timeout.restype = ctypes.c_int
        lib.flowmm_decode_workspace_bytes.restype = ctypes.c_int
        lib.flowmm_decode_attention.restype = ctypes.c_int
        lib.flowmm_full_flow_workspace_bytes.restype = ctypes.c_int
        lib.flowmm_full_flow.restype = ctypes.c_int
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().flowmm_status_string(ctypes.c_int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise FlowmmError(code, where)


def _p(t: Optional[torch.Tensor]):
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda:
        raise ValueError("flowmm takes CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def torch_dtype(code: int):
    return torch.bfloat16 if code == BF16 else torch.float32


def flowmm_workspace_bytes(p: Params) -> int:
    n = ctypes.c_size_t(0)
    cp = p.c()
    _check(load().flowmm_workspace_bytes(ctypes.byref(cp), ctypes.byref(n)), "flowmm_workspace_bytes")
    return int(n.value)


def alloc_workspace(p: Params, device="cuda") -> torch.Tensor:
    """A workspace of the required size with its status word cleared."""
    ws = torch.empty(flowmm_workspace_bytes(p), dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def flowmm_score(p: Params, q_win, k, modality, importance, cross_mass, ws):
    cp = p.c(q=q_win, k=k)
    _check(load().flowmm_score(ctypes.byref(cp), _p(q_win), _p(k), _p(modality), _p(importance), _p(cross_mass),
                               _p(ws), ctypes.c_size_t(ws.numel()), _stream()), "flowmm_score")


def flowmm_full_flow_workspace_bytes(p: Params) -> int:
    n = ctypes.c_size_t(0)
    cp = p.c()
    _check(load().flowmm_full_flow_workspace_bytes(ctypes.byref(cp), ctypes.byref(n)), "flowmm_full_flow_workspace_bytes")
    return int(n.value)


def flowmm_full_flow(p: Params, q_full, k, modality, cross_mass, rho, strategy, ws):
    """Eq. 6 and Eq. 7 over every query row of the prefill: q_full [units, q_heads, seq_len, head_dim]."""
    if q_full.dim() != 4 or q_full.stride(3) != 1:
        raise ValueError("expected a [units, heads, tokens, head_dim] tensor with contiguous head_dim")
    cp = p.c(k=k)
    qs = (ctypes.c_int64 * 3)(q_full.stride(0), q_full.stride(1), q_full.stride(2))
    _check(load().flowmm_full_flow(ctypes.byref(cp), _p(q_full), qs, _p(k), _p(modality), _p(cross_mass), _p(rho),
                                   _p(strategy), _p(ws), ctypes.c_size_t(ws.numel()), _stream()), "flowmm_full_flow")


def flowmm_layer_flow(p: Params, cross_mass, rho, strategy):
    cp = p.c()
    _check(load().flowmm_layer_flow(ctypes.byref(cp), _p(cross_mass), _p(rho), _p(strategy), _stream()),
           "flowmm_layer_flow")


def flowmm_select(p: Params, importance, retained_idx, evicted_idx, ws):
    cp = p.c()
    _check(load().flowmm_select(ctypes.byref(cp), _p(importance), _p(retained_idx), _p(evicted_idx), _p(ws),
                                ctypes.c_size_t(ws.numel()), _stream()), "flowmm_select")


def flowmm_match(p: Params, k, importance, modality, retained_idx, evicted_idx, strategy, match, match_sim, ws):
    cp = p.c(k=k)
    _check(load().flowmm_match(ctypes.byref(cp), _p(k), _p(importance), _p(modality), _p(retained_idx),
                               _p(evicted_idx), _p(strategy), _p(match), _p(match_sim), _p(ws),
                               ctypes.c_size_t(ws.numel()), _stream()), "flowmm_match")


def flowmm_merge(p: Params, k, v, retained_idx, evicted_idx, match, match_sim, k_out, v_out, ws):
    cp = p.c(k=k, v=v, ko=k_out, vo=v_out)
    _check(load().flowmm_merge(ctypes.byref(cp), _p(k), _p(v), _p(retained_idx), _p(evicted_idx), _p(match),
                               _p(match_sim), _p(k_out), _p(v_out), _p(ws), ctypes.c_size_t(ws.numel()), _stream()),
           "flowmm_merge")


def flowmm_merge_static(p: Params, k, v, retained_idx, evicted_idx, match, match_sim, k_out, v_out):
    """flowmm_merge for callers that cannot allocate: no workspace argument, the scratch is a
    fixed array inside the library (see include/flowmm.h for its size limit and sharing rules)."""
    cp = p.c(k=k, v=v, ko=k_out, vo=v_out)
    _check(load().flowmm_merge_static(ctypes.byref(cp), _p(k), _p(v), _p(retained_idx), _p(evicted_idx), _p(match),
                                      _p(match_sim), _p(k_out), _p(v_out), _stream()), "flowmm_merge_static")


def flowmm_merge_static_status() -> int:
    """Device status of the flowmm_merge_static calls since the last read (0 = ok); waits for the stream, clears."""
    return int(load().flowmm_merge_static_status(_stream()))


def flowmm_merge_static_poke_status(word: int):
    _check(load().flowmm_merge_static_poke_status(ctypes.c_int32(word), _stream()), "flowmm_merge_static_poke_status")


def flowmm_compress_layer(p: Params, q_win, k, v, modality, k_out, v_out, ws, importance=None, rho=None,
                          strategy=None, retained_idx=None, evicted_idx=None, match=None, match_sim=None):
    cp = p.c(q=q_win, k=k, v=v, ko=k_out, vo=v_out)
    _check(load().flowmm_compress_layer(ctypes.byref(cp), _p(q_win), _p(k), _p(v), _p(modality), _p(k_out),
                                        _p(v_out), _p(importance), _p(rho), _p(strategy), _p(retained_idx),
                                        _p(evicted_idx), _p(match), _p(match_sim), _p(ws),
                                        ctypes.c_size_t(ws.numel()), _stream()), "flowmm_compress_layer")


def flowmm_recompress_workspace_bytes(p: Params) -> int:
    n = ctypes.c_size_t(0)
    cp = p.c()
    _check(load().flowmm_recompress_workspace_bytes(ctypes.byref(cp), ctypes.byref(n)), "flowmm_recompress_workspace_bytes")
    return int(n.value)


def flowmm_recompress(p: Params, q_win, k_cache, v_cache, row_modality, k_out, v_out, row_modality_out, ws,
                      importance=None, rho=None, strategy=None, retained_idx=None, evicted_idx=None, match=None,
                      match_sim=None):
    """Section 3.3 again on a cache that grew during decoding; row_modality [units, kv_heads, rows] uint8."""
    cp = p.c(q=q_win, k=k_cache, v=v_cache, ko=k_out, vo=v_out)
    _check(load().flowmm_recompress(ctypes.byref(cp), _p(q_win), _p(k_cache), _p(v_cache), _p(row_modality), _p(k_out),
                                    _p(v_out), _p(row_modality_out), _p(importance), _p(rho), _p(strategy),
                                    _p(retained_idx), _p(evicted_idx), _p(match), _p(match_sim), _p(ws),
                                    ctypes.c_size_t(ws.numel()), _stream()), "flowmm_recompress")


def flowmm_last_device_status(ws) -> int:
    return int(load().flowmm_last_device_status(_p(ws), _stream()))


class _CDecodeParams(ctypes.Structure):
    _fields_ = [
        ("n_units", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("n_keys", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("path", ctypes.c_int32),
        ("k_stride", ctypes.c_int64 * 3), ("v_stride", ctypes.c_int64 * 3),
    ]


def _decode_params(q, k, v, softmax_scale: float, path: int) -> _CDecodeParams:
    if q.dim() != 3 or not q.is_contiguous():
        raise ValueError("q must be a contiguous [units, q_heads, head_dim] tensor")
    if k.dim() != 4 or v.dim() != 4 or k.stride(3) != 1 or v.stride(3) != 1 or k.shape != v.shape:
        raise ValueError("k, v must be [units, kv_heads, keys, head_dim] tensors with contiguous head_dim")
    dtype = BF16 if q.dtype == torch.bfloat16 else F32
    cp = _CDecodeParams(q.shape[0], q.shape[1], k.shape[1], q.shape[2], k.shape[2], dtype, softmax_scale, path)
    cp.k_stride = (ctypes.c_int64 * 3)(k.stride(0), k.stride(1), k.stride(2))
    cp.v_stride = (ctypes.c_int64 * 3)(v.stride(0), v.stride(1), v.stride(2))
    return cp


def flowmm_decode_workspace_bytes(q, k, v, softmax_scale: float = 0.0, path: int = PATH_AUTO) -> int:
    n = ctypes.c_size_t(0)
    cp = _decode_params(q, k, v, softmax_scale, path)
    _check(load().flowmm_decode_workspace_bytes(ctypes.byref(cp), ctypes.byref(n)), "flowmm_decode_workspace_bytes")
    return int(n.value)


def flowmm_decode_attention(q, k, v, out, ws, softmax_scale: float = 0.0, path: int = PATH_AUTO):
    """Eq. 4 for one new query per head over the cache rows of k, v; out [units, q_heads, head_dim] float32."""
    cp = _decode_params(q, k, v, softmax_scale, path)
    _check(load().flowmm_decode_attention(ctypes.byref(cp), _p(q), _p(k), _p(v), _p(out), _p(ws),
                                          ctypes.c_size_t(ws.numel()), _stream()), "flowmm_decode_attention")


def flowmm_selftest_wait_timeout(ws):
    """Enqueue the kernel whose wait runs out; flowmm_last_device_status(ws) then reports TIMEOUT (8)."""
    _check(load().flowmm_selftest_wait_timeout(_p(ws), _stream()), "flowmm_selftest_wait_timeout")


def flowmm_debug_build() -> bool:
    return bool(load().flowmm_debug_build())


def flowmm_last_launch_count() -> int:
    return int(load().flowmm_last_launch_count())


def flowmm_profile_enable(on: bool):
    _check(load().flowmm_profile_enable(ctypes.c_int32(1 if on else 0)), "flowmm_profile_enable")


def flowmm_profile_read(max_entries: int = 32):
    """[(kernel name, milliseconds), ...] of the most recent entry point, in launch order."""
    names = (ctypes.c_char_p * max_entries)()
    ms = (ctypes.c_float * max_entries)()
    n = load().flowmm_profile_read(names, ms, ctypes.c_int32(max_entries))
    if n < 0:
        raise FlowmmError(7, "flowmm_profile_read")
    return [(names[i].decode(), float(ms[i])) for i in range(n)]


def compress_layer_alloc(p: Params, q_win, k, v, modality, ws=None, diagnostics=True):
    """Allocate the outputs (and optionally every intermediate) and run flowmm_compress_layer.
    Returns a dict of tensors.  Allocation only; the computation is the C call."""
    dev = k.device
    U, Hq, Hkv, L, B, E, D = p.n_units, p.n_q_heads, p.n_kv_heads, p.seq_len, p.n_keep, p.n_evict, p.head_dim
    if ws is None:
        ws = alloc_workspace(p, dev)
    out = {
        "k_out": torch.empty((U, Hkv, B, D), dtype=k.dtype, device=dev),
        "v_out": torch.empty((U, Hkv, B, D), dtype=v.dtype, device=dev),
    }
    if diagnostics:
        out.update({
            "importance": torch.empty((U, Hkv, L), dtype=torch.float32, device=dev),
            "rho": torch.empty((U,), dtype=torch.float32, device=dev),
            "strategy": torch.empty((U,), dtype=torch.int32, device=dev),
            "retained": torch.empty((U, Hkv, B), dtype=torch.int32, device=dev),
            "evicted": torch.empty((U, Hkv, E), dtype=torch.int32, device=dev),
            "match": torch.empty((U, Hkv, E), dtype=torch.int32, device=dev),
            "match_sim": torch.empty((U, Hkv, E), dtype=torch.float32, device=dev),
        })
    flowmm_compress_layer(p, q_win, k, v, modality, out["k_out"], out["v_out"], ws,
                          out.get("importance"), out.get("rho"), out.get("strategy"), out.get("retained"),
                          out.get("evicted"), out.get("match"), out.get("match_sim"))
    out["ws"] = ws
    return out
