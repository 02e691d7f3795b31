"""Cross-modal interaction ratio over every query row of the prefill (Eq. 6 and Eq. 7 taken literally) on the
GPU against the oracle's scoring step with the whole prompt as the window."""
import numpy as np
import pytest
import torch

from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

from gpu_util import to_dev

pytestmark = pytest.mark.gpu


def _oracle(U, Hq, Hkv, D, L, q, k, m, theta):
    p = O.OracleParams(U, Hq, Hkv, D, L, L, 1, theta=theta)           # window = the whole prompt: every row is a proxy row
    _, cross, total = O.score(p, q, k, m)
    rho, strat = O.layer_flow(p, cross, total)
    return cross, rho, strat


def _gpu(U, Hq, Hkv, D, L, q, k, m, theta, dtype):
    fp = F.Params(U, Hq, Hkv, D, L, 1, 1, dtype=dtype, theta=theta)
    qd, kd = to_dev(q, dtype), to_dev(k, dtype)
    md = torch.from_numpy(np.ascontiguousarray(m, dtype=np.uint8)).cuda()
    cross = torch.full((U, Hq), float("nan"), device="cuda")
    rho = torch.full((U,), float("nan"), device="cuda")
    strat = torch.full((U,), -7, dtype=torch.int32, device="cuda")
    ws = torch.zeros(F.flowmm_full_flow_workspace_bytes(fp), dtype=torch.uint8, device="cuda")
    F.flowmm_full_flow(fp, qd, kd, md, cross, rho, strat, ws)
    assert F.flowmm_last_device_status(ws) == 0
    return cross.cpu().numpy().astype(np.float64), rho.cpu().numpy().astype(np.float64), strat.cpu().numpy()


@pytest.mark.parametrize("dtype,D", [(F.BF16, 128), (F.F32, 64), (F.BF16, 64)])
def test_ragged_lengths_against_oracle(dtype, D):
    rng = np.random.default_rng(5 + D + dtype)
    for (U, Hq, Hkv, L) in [(2, 4, 2, 300), (1, 7, 1, 128), (1, 2, 2, 45), (2, 2, 1, 513)]:
        q = rng.standard_normal((U, Hq, L, D)).astype(np.float32)
        k = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
        m = (rng.random((U, L)) < 0.6).astype(np.uint8)
        if dtype == F.BF16:
            q, k = inputs.round_to_bf16(q), inputs.round_to_bf16(k)
        cross, rho, strat = _oracle(U, Hq, Hkv, D, L, q, k, m, 0.35)
        g_cross, g_rho, g_strat = _gpu(U, Hq, Hkv, D, L, q, k, m, 0.35, dtype)
        assert np.allclose(g_cross, cross, rtol=1e-3, atol=1e-6 * L), (U, Hq, Hkv, L)     # masses within 1e-3 relative
        assert np.allclose(g_rho, rho, atol=1e-4), (g_rho, rho)
        decided = np.abs(rho - 0.35) > 1e-4                            # away from the threshold the rule must agree
        assert np.array_equal(g_strat[decided], strat[decided])


def test_single_modality_has_no_cross_flow_and_workload_stack_is_finite():
    rng = np.random.default_rng(9)
    U, Hq, Hkv, D, L = 1, 2, 2, 128, 200
    q = inputs.round_to_bf16(rng.standard_normal((U, Hq, L, D)).astype(np.float32))
    k = inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32))
    for vis in (0, 1):
        cross, rho, strat = _gpu(U, Hq, Hkv, D, L, q, k, np.full((U, L), vis, np.uint8), 0.25, F.BF16)
        assert np.all(cross == 0.0) and np.all(rho == 0.0) and np.all(strat == 0)
    # a stack of the cfg2 workload: keys of the workload, queries drawn like its window queries
    wl = configs.get("cfg2")
    units = [(l, 0) for l in (0, 15, 31)]
    _, kd, _, md = inputs.make_stack_device(wl, "cuda", units)
    qd = torch.randn((3, wl.n_q_heads, wl.seq_len, wl.head_dim), device="cuda").to(torch.bfloat16)
    cross, rho, strat = _oracle(3, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, qd.float().cpu().numpy(),
                                kd.float().cpu().numpy(), md.cpu().numpy(), wl.theta)
    g = _gpu(3, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, qd.float().cpu().numpy(), kd.float().cpu().numpy(),
             md.cpu().numpy(), wl.theta, F.BF16)
    assert np.allclose(g[1], rho, atol=1e-4)


def test_video_shaped_prompt_at_full_length():
    """One KV head with its seven query heads at the multi-image workload's shape: 8 448 tokens, eight frames of
    1 024 visual tokens interleaved with text, keys of the workload's generator (frame-correlated), queries drawn
    with a modality-dependent offset so that both cross terms are substantial.  66 query tiles, the long-context
    tensor-core path."""
    wl = configs.get("cfg4")
    L, D, G = wl.seq_len, wl.head_dim, wl.group
    unit = inputs.make_unit(wl, 20, 0)
    k = unit["k"][:1][None]                                            # [1, 1, L, D], already bf16 values
    m = unit["modality"][None]
    rng = np.random.default_rng(77)
    sign = np.where(m[0] == 1, -1.0, 1.0).astype(np.float32)
    q = rng.standard_normal((1, G, L, D)).astype(np.float32) + (-3.0 / np.sqrt(D)) * sign[None, None, :, None]
    q = inputs.round_to_bf16(q)
    cross, rho, strat = _oracle(1, G, 1, D, L, q, k, m, wl.theta)
    g_cross, g_rho, g_strat = _gpu(1, G, 1, D, L, q, k, m, wl.theta, F.BF16)
    assert cross.min() > 1.0                                           # a real cross-modal mass on every head
    assert np.allclose(g_cross, cross, rtol=1e-3, atol=0.0), np.abs(g_cross / cross - 1).max()
    assert np.allclose(g_rho, rho, atol=1e-4)
    if abs(rho[0] - wl.theta) > 1e-4:
        assert g_strat[0] == strat[0]
