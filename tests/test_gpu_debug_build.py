"""The build with index checks (-DFLOWMM_DEBUG) in place of a memory checker: same results as the release
build on good inputs, nothing written outside the buffers it was given (guard regions around every output
and around the workspace), and bad index lists reported as FLOWMM_ERR_INDEX instead of being followed."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import compare as C
from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import build, configs, inputs

from gpu_util import gpu_params, oracle_params, to_dev

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


@pytest.fixture()
def debug_lib(monkeypatch):
    """The binding pointed at libflowmm_debug.so for the duration of a test."""
    path = build.build(debug=True)
    release = F.load()
    monkeypatch.setattr(F, "_lib", None)
    monkeypatch.setattr(F, "LIB_PATH", path)
    lib = F.load()
    assert F.flowmm_debug_build() and lib is not release
    yield lib


class Guarded:
    """A tensor inside a larger byte buffer whose margins hold a pattern that must survive."""

    def __init__(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((GUARD + n + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(shape)

    def intact(self):
        return bool((self.raw[:GUARD] == PATTERN).all() and (self.raw[-GUARD:] == PATTERN).all())


def _run_guarded(p, data, dtype):
    fp = gpu_params(p, dtype)
    U, Hkv, L, B, E, D = p.n_units, p.n_kv_heads, p.seq_len, p.n_keep, p.seq_len - p.n_keep, p.head_dim
    tdt = F.torch_dtype(dtype)
    bufs = {
        "k_out": Guarded((U, Hkv, B, D), tdt), "v_out": Guarded((U, Hkv, B, D), tdt),
        "importance": Guarded((U, Hkv, L), torch.float32), "rho": Guarded((U,), torch.float32),
        "strategy": Guarded((U,), torch.int32), "retained": Guarded((U, Hkv, B), torch.int32),
        "evicted": Guarded((U, Hkv, max(E, 1)), torch.int32), "match": Guarded((U, Hkv, max(E, 1)), torch.int32),
        "match_sim": Guarded((U, Hkv, max(E, 1)), torch.float32),
        "ws": Guarded((F.flowmm_workspace_bytes(fp),), torch.uint8),
    }
    bufs["ws"].t[:256].zero_()
    q, k, v = (to_dev(data[x], dtype) for x in "qkv")
    m = torch.from_numpy(np.ascontiguousarray(data["modality"])).cuda()
    t = {key: b.t for key, b in bufs.items()}
    F.flowmm_compress_layer(fp, q, k, v, m, t["k_out"], t["v_out"], t["ws"], t["importance"], t["rho"], t["strategy"],
                            t["retained"], t["evicted"], t["match"], t["match_sim"])
    assert F.flowmm_last_device_status(t["ws"]) == 0
    for key, b in bufs.items():
        assert b.intact(), "guard region around %s was written" % key
    return {key: (b.t.float().cpu().numpy().astype(np.float64) if b.t.is_floating_point() else b.t.cpu().numpy())
            for key, b in bufs.items() if key != "ws"}


def test_small_fp32_workload_with_guards(debug_lib):
    wl = configs.get("cfg1")
    data = inputs.make_units(wl, [(0, 0)])
    p = oracle_params(wl, 1, 250)
    g = _run_guarded(p, data, F.F32)
    C.compare(p, data["q"], data["k"], data["v"], data["modality"], g, bf16_out=False)


@pytest.mark.parametrize("shape", [(2, 6, 2, 128, 333, 21, 37), (1, 4, 2, 128, 1031, 32, 300), (1, 8, 1, 128, 2600, 64, 500)])
def test_ragged_bf16_cases_with_guards(debug_lib, shape):
    U, Hq, Hkv, D, L, W, B = shape
    rng = np.random.default_rng(L)
    data = {"q": inputs.round_to_bf16(rng.standard_normal((U, Hq, W, D)).astype(np.float32)),
            "k": inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32)),
            "v": inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32)),
            "modality": (rng.random((U, L)) < 0.6).astype(np.uint8)}
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, theta=0.5, tau=3.0, tau_mode=O.TAU_REL)
    g = _run_guarded(p, data, F.BF16)
    C.compare(p, data["q"], data["k"], data["v"], data["modality"], g, bf16_out=True)


def test_bad_index_lists_are_reported_not_followed(debug_lib):
    rng = np.random.default_rng(8)
    U, Hq, Hkv, D, L, W, B = 1, 2, 2, 128, 400, 16, 50
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, tau=3.0, tau_mode=O.TAU_REL)
    fp = gpu_params(p, F.BF16)
    q = to_dev(inputs.round_to_bf16(rng.standard_normal((U, Hq, W, D)).astype(np.float32)), F.BF16)
    k = to_dev(inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32)), F.BF16)
    v = to_dev(inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32)), F.BF16)
    m = torch.from_numpy((rng.random((U, L)) < 0.5).astype(np.uint8)).cuda()
    good = F.compress_layer_alloc(fp, q, k, v, m)
    assert F.flowmm_last_device_status(good["ws"]) == 0
    out = Guarded((U, Hkv, B, D), torch.bfloat16)
    vout = Guarded((U, Hkv, B, D), torch.bfloat16)
    before = out.raw.clone()
    for which, value in (("retained", L + 7), ("evicted", -3), ("match", B)):
        lists = {key: good[key].clone() for key in ("retained", "evicted", "match")}
        lists[which][0, 1, 5] = value
        with pytest.raises(F.FlowmmError) as e:
            F.flowmm_merge(fp, k, v, lists["retained"], lists["evicted"], lists["match"], good["match_sim"], out.t, vout.t,
                           good["ws"])
        assert e.value.code == 10, which
        assert F.flowmm_last_launch_count() == 0
        assert F.flowmm_last_device_status(good["ws"]) == 10          # recorded in the status word too, and cleared by the read
        assert torch.equal(out.raw, before) and vout.intact()
    # the untouched lists still merge, and give what the fused call gave
    F.flowmm_merge(fp, k, v, good["retained"], good["evicted"], good["match"], good["match_sim"], out.t, vout.t, good["ws"])
    assert F.flowmm_last_device_status(good["ws"]) == 0
    assert torch.equal(out.t, good["k_out"]) and torch.equal(vout.t, good["v_out"]) and out.intact() and vout.intact()
