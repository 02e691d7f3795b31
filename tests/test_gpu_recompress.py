"""flowmm_recompress (Section 3.3 again on a cache that grew by Eq. 3) against the oracle's recompress()."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import compare as C
from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import inputs

from gpu_util import gpu_params, to_dev

pytestmark = pytest.mark.gpu


def _grown_cache(rng, U, Hq, Hkv, D, L, W, B, T, dtype):
    """A prompt compressed once on the GPU, then T decoded (text) rows appended to every head's cache."""
    rnd = lambda *shape: rng.standard_normal(shape).astype(np.float32)
    q, k, v = rnd(U, Hq, W, D), rnd(U, Hkv, L, D), rnd(U, Hkv, L, D)
    k_new, v_new, q2 = rnd(U, Hkv, T, D), rnd(U, Hkv, T, D), rnd(U, Hq, W, D)
    if dtype == F.BF16:
        q, k, v, k_new, v_new, q2 = (inputs.round_to_bf16(x) for x in (q, k, v, k_new, v_new, q2))
    m = (rng.random((U, L)) < 0.6).astype(np.uint8)
    fp = F.Params(U, Hq, Hkv, D, L, W, B, dtype=dtype, theta=0.4, tau=3.0, tau_mode=F.TAU_REL)
    first = F.compress_layer_alloc(fp, to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype), torch.from_numpy(m).cuda())
    assert F.flowmm_last_device_status(first["ws"]) == 0
    ret = first["retained"].cpu().numpy()
    k_cache = np.concatenate([first["k_out"].float().cpu().numpy(), k_new], axis=2)
    v_cache = np.concatenate([first["v_out"].float().cpu().numpy(), v_new], axis=2)
    rm = np.concatenate([np.take_along_axis(np.repeat(m[:, None, :], Hkv, axis=1), ret.astype(np.int64), -1),
                         np.zeros((U, Hkv, T), np.uint8)], axis=2)
    return q2, k_cache, v_cache, rm


def _run(p: O.OracleParams, q, k, v, rm, dtype, path=F.PATH_AUTO):
    fp = gpu_params(p, dtype, path)
    U, Hkv, L, B, E, D = p.n_units, p.n_kv_heads, p.seq_len, p.n_keep, p.seq_len - p.n_keep, p.head_dim
    qd, kd, vd = to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype)
    rmd = torch.from_numpy(rm).cuda()
    tdt = F.torch_dtype(dtype)
    out = {
        "k_out": torch.empty((U, Hkv, B, D), dtype=tdt, device="cuda"), "v_out": torch.empty((U, Hkv, B, D), dtype=tdt, device="cuda"),
        "row_modality_out": torch.full((U, Hkv, B), 9, dtype=torch.uint8, device="cuda"),
        "importance": torch.empty((U, Hkv, L), device="cuda"), "rho": torch.empty((U,), device="cuda"),
        "strategy": torch.empty((U,), dtype=torch.int32, device="cuda"),
        "retained": torch.empty((U, Hkv, B), dtype=torch.int32, device="cuda"),
        "evicted": torch.empty((U, Hkv, E), dtype=torch.int32, device="cuda"),
        "match": torch.empty((U, Hkv, E), dtype=torch.int32, device="cuda"),
        "match_sim": torch.empty((U, Hkv, E), device="cuda"),
    }
    ws = torch.zeros(F.flowmm_recompress_workspace_bytes(fp), dtype=torch.uint8, device="cuda")
    F.flowmm_recompress(fp, qd, kd, vd, rmd, out["k_out"], out["v_out"], out["row_modality_out"], ws,
                        out["importance"], out["rho"], out["strategy"], out["retained"], out["evicted"], out["match"],
                        out["match_sim"])
    assert F.flowmm_last_device_status(ws) == 0
    return {key: (t.float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy()) for key, t in out.items()}


def _check(p: O.OracleParams, q, k, v, rm, dtype, path=F.PATH_AUTO):
    g = _run(p, q, k, v, rm, dtype, path)
    ref = O.recompress(p, q, k, v, rm)
    U, Hq, Hkv, D, L, W, B = p.n_units, p.n_q_heads, p.n_kv_heads, p.head_dim, p.seq_len, p.window, p.n_keep
    G = Hq // Hkv
    # the layer's rho and its one strategy
    assert np.allclose(g["rho"], ref["rho"], rtol=1e-3, atol=1e-7)
    decided = np.abs(ref["rho"] - p.theta) > 1e-4 * p.theta
    assert np.array_equal(g["strategy"][decided], ref["strategy"][decided])
    assert np.array_equal(g["row_modality_out"], np.take_along_axis(rm, g["retained"].astype(np.int64), -1))
    # everything else head by head: each (unit, KV head) is a problem of its own under the layer's strategy
    for u in range(U):
        forced = O.FLOW_FORCE_CROSS if g["strategy"][u] == O.CROSS else O.FLOW_FORCE_INTRA
        ph = dataclasses.replace(p, n_units=Hkv, n_q_heads=G, n_kv_heads=1, flow_mode=forced)
        qh, kh, vh, mh = q[u].reshape(Hkv, G, W, D), k[u].reshape(Hkv, 1, L, D), v[u].reshape(Hkv, 1, L, D), rm[u]
        _, cross, total = O.score(ph, qh, kh, mh)
        gh = {key: g[key][u].reshape((Hkv, 1) + g[key].shape[2:]) for key in
              ("importance", "retained", "evicted", "match", "match_sim", "k_out", "v_out")}
        gh["rho"] = O.layer_flow(ph, cross, total)[0]           # (per-head shares; the layer's rho was checked above)
        gh["strategy"] = np.full(Hkv, g["strategy"][u], np.int32)
        C.compare(ph, qh, kh, vh, mh, gh, bf16_out=dtype == F.BF16)
    return g


@pytest.mark.parametrize("dtype,D,path", [(F.BF16, 128, F.PATH_AUTO), (F.BF16, 128, F.PATH_SIMT), (F.F32, 64, F.PATH_AUTO)])
def test_second_round_against_oracle(dtype, D, path):
    rng = np.random.default_rng(40 + D + path)
    for (U, Hq, Hkv, L, W, B, T, B2) in [(2, 4, 2, 300, 16, 60, 24, 40), (1, 6, 2, 900, 32, 300, 40, 120)]:
        q2, k_cache, v_cache, rm = _grown_cache(rng, U, Hq, Hkv, D, L, W, B, T, dtype)
        p = O.OracleParams(U, Hq, Hkv, D, B + T, W, B2, theta=0.3, tau=3.0, tau_mode=O.TAU_REL)
        g = _check(p, q2, k_cache, v_cache, rm, dtype, path)
        assert g["k_out"].shape == (U, Hkv, B2, D)


def test_long_cache_on_the_general_tensor_core_kernels():
    # 2 500 cache rows, 400 kept: two-pass scoring, the general matching kernel and the gather merge, with row
    # modalities that differ between the heads of a unit
    rng = np.random.default_rng(77)
    q2, k_cache, v_cache, rm = _grown_cache(rng, 1, 8, 2, 128, 4000, 64, 2436, 64, F.BF16)
    p = O.OracleParams(1, 8, 2, 128, 2500, 64, 400, theta=0.3, tau=4.0, tau_mode=O.TAU_REL)
    assert not np.array_equal(rm[0, 0], rm[0, 1])
    _check(p, q2, k_cache, v_cache, rm, F.BF16)


def test_full_budget_returns_the_cache_with_its_appended_rows():
    rng = np.random.default_rng(5)
    q2, k_cache, v_cache, rm = _grown_cache(rng, 2, 4, 2, 128, 200, 8, 30, 10, F.BF16)
    p = O.OracleParams(2, 4, 2, 128, 40, 8, 40)
    g = _run(p, q2, k_cache, v_cache, rm, F.BF16)
    assert np.array_equal(g["k_out"], k_cache.astype(np.float64)) and np.array_equal(g["v_out"], v_cache.astype(np.float64))
    assert np.array_equal(g["row_modality_out"], rm)


def test_strided_units_are_refused():
    fp = F.Params(2, 4, 2, 128, 64, 8, 16, dtype=F.BF16)
    k = torch.zeros((2, 3, 64, 128), dtype=torch.bfloat16, device="cuda")[:, :2]       # unit stride != heads x head stride
    q = torch.zeros((2, 4, 8, 128), dtype=torch.bfloat16, device="cuda")
    rm = torch.zeros((2, 2, 64), dtype=torch.uint8, device="cuda")
    ko = torch.zeros((2, 2, 16, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(F.flowmm_recompress_workspace_bytes(fp), dtype=torch.uint8, device="cuda")
    with pytest.raises(F.FlowmmError) as e:
        F.flowmm_recompress(fp, q, k, k, rm, ko, torch.zeros_like(ko), torch.zeros((2, 2, 16), dtype=torch.uint8, device="cuda"), ws)
    assert e.value.code == 6
