"""Stepwise entry points and host-side error behaviour of the C ABI, on a GPU."""
import numpy as np
import pytest
import torch

from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

from gpu_util import gpu_params, oracle_params, to_dev

pytestmark = pytest.mark.gpu


def test_stepwise_equals_fused_call():
    wl = configs.get("cfg3")
    data = inputs.make_units(wl, [(13, 0), (14, 0)])
    p = oracle_params(wl, 2, 100)
    fp = gpu_params(p, F.BF16)
    q, k, v = (to_dev(data[x], F.BF16) for x in "qkv")
    m = torch.from_numpy(data["modality"]).cuda()
    full = F.compress_layer_alloc(fp, q, k, v, m)
    U, Hq, Hkv, L, B, E, D = fp.n_units, fp.n_q_heads, fp.n_kv_heads, fp.seq_len, fp.n_keep, fp.n_evict, fp.head_dim
    ws = F.alloc_workspace(fp)
    dev = "cuda"
    imp = torch.empty((U, Hkv, L), device=dev); cross = torch.empty((U, Hq), device=dev)
    rho = torch.empty((U,), device=dev); strat = torch.empty((U,), dtype=torch.int32, device=dev)
    ret = torch.empty((U, Hkv, B), dtype=torch.int32, device=dev); evi = torch.empty((U, Hkv, E), dtype=torch.int32, device=dev)
    mt = torch.empty((U, Hkv, E), dtype=torch.int32, device=dev); sim = torch.empty((U, Hkv, E), device=dev)
    ko = torch.empty((U, Hkv, B, D), dtype=torch.bfloat16, device=dev); vo = torch.empty_like(ko)
    F.flowmm_score(fp, q, k, m, imp, cross, ws)
    F.flowmm_layer_flow(fp, cross, rho, strat)
    F.flowmm_select(fp, imp, ret, evi, ws)
    F.flowmm_match(fp, k, imp, m, ret, evi, strat, mt, sim, ws)
    F.flowmm_merge(fp, k, v, ret, evi, mt, sim, ko, vo, ws)
    assert F.flowmm_last_device_status(ws) == 0
    for name, t in (("importance", imp), ("rho", rho), ("strategy", strat), ("retained", ret), ("evicted", evi),
                    ("match", mt), ("match_sim", sim), ("k_out", ko), ("v_out", vo)):
        assert torch.equal(t, full[name]), name
    # Eq. 6 from the per-head masses the score step returned
    assert np.allclose(rho.cpu().numpy(), (cross.cpu().numpy() / fp.window).mean(1), rtol=1e-6)


def test_errors_are_reported_not_computed():
    fp = F.Params(1, 4, 2, 128, 64, 8, 16, dtype=F.BF16)
    q = torch.zeros((1, 4, 8, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((1, 2, 64, 128), dtype=torch.bfloat16, device="cuda")
    m = torch.zeros((1, 64), dtype=torch.uint8, device="cuda")
    imp = torch.zeros((1, 2, 64), device="cuda"); cross = torch.zeros((1, 4), device="cuda")
    ws = F.alloc_workspace(fp)
    with pytest.raises(F.FlowmmError) as e:
        F.flowmm_score(fp, q, k, m, imp, cross, ws[:1024])
    assert e.value.code == 5
    with pytest.raises(F.FlowmmError) as e:
        F.flowmm_score(fp, q, None, m, imp, cross, ws)
    assert e.value.code == 1
    with pytest.raises(F.FlowmmError) as e:
        F.flowmm_score(fp, q, k, m, imp, cross, ws[8:])
    assert e.value.code == 6
    flat = torch.zeros(k.numel() + 8, dtype=torch.bfloat16, device="cuda")
    k_odd = flat[1:1 + k.numel()].view(k.shape)              # 2 bytes off a 16-byte boundary
    with pytest.raises(F.FlowmmError) as e:
        F.flowmm_score(fp, q, k_odd, m, imp, cross, ws)
    assert e.value.code == 6
    F.flowmm_score(fp, q, k, m, imp, cross, ws)
    assert F.flowmm_last_launch_count() >= 1
    torch.cuda.synchronize()


def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    """No kernel here can hang the GPU: a wait nothing satisfies gives up after its limit, the status
    word says so, and the next call works as if nothing had happened."""
    fp = F.Params(1, 4, 2, 128, 300, 32, 30, dtype=F.BF16)
    ws = F.alloc_workspace(fp)
    F.flowmm_selftest_wait_timeout(ws)
    assert F.flowmm_last_device_status(ws) == 8            # FLOWMM_ERR_TIMEOUT
    assert F.flowmm_last_device_status(ws) == 0            # reading it cleared it
    rng = np.random.default_rng(5)
    q = to_dev(inputs.round_to_bf16(rng.standard_normal((1, 4, 32, 128)).astype(np.float32)), F.BF16)
    k = to_dev(inputs.round_to_bf16(rng.standard_normal((1, 2, 300, 128)).astype(np.float32)), F.BF16)
    v = to_dev(inputs.round_to_bf16(rng.standard_normal((1, 2, 300, 128)).astype(np.float32)), F.BF16)
    m = torch.from_numpy((rng.random((1, 300)) < 0.5).astype(np.uint8)).cuda()
    out = F.compress_layer_alloc(fp, q, k, v, m, ws=ws)
    assert F.flowmm_last_device_status(ws) == 0
    assert torch.isfinite(out["k_out"].float()).all()
