"""Decode-step attention over a cache (Eq. 4) on the GPU against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

from gpu_util import oracle_params, to_dev

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-4, 1e-4      # fp32 accumulation of exact bf16 products, 2^-22 exponentials, weights kept to 2^-17


def _run(q, k, v, dtype, scale=0.0, path=F.PATH_AUTO):
    qd, kd, vd = to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype)
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(F.flowmm_decode_workspace_bytes(qd, kd, vd, scale, path), dtype=torch.uint8, device="cuda")
    F.flowmm_decode_attention(qd, kd, vd, out, ws, scale, path)
    assert F.flowmm_last_device_status(ws) == 0
    return out.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("dtype", [F.F32, F.BF16])
@pytest.mark.parametrize("D", [64, 128])
def test_ragged_shapes_against_oracle(dtype, D):
    rng = np.random.default_rng(40 + D + dtype)
    for (U, Hq, Hkv, N) in [(2, 6, 2, 333), (1, 8, 1, 1031), (3, 4, 4, 65), (1, 7, 1, 1), (2, 2, 2, 5000)]:
        q = rng.standard_normal((U, Hq, D)).astype(np.float32)
        k = rng.standard_normal((U, Hkv, N, D)).astype(np.float32)
        v = rng.standard_normal((U, Hkv, N, D)).astype(np.float32)
        if dtype == F.BF16:
            q, k, v = inputs.round_to_bf16(q), inputs.round_to_bf16(k), inputs.round_to_bf16(v)
        ref = O.decode_attention(q, k, v)
        for path in (F.PATH_AUTO, F.PATH_SIMT):          # AUTO is the tensor-core kernel for bf16 at head_dim 128
            got = _run(q, k, v, dtype, path=path)
            assert np.allclose(got, ref, rtol=RTOL, atol=ATOL), (U, Hq, Hkv, N, path, np.abs(got - ref).max())


def test_peaked_attention_and_explicit_scale():
    rng = np.random.default_rng(9)
    q = inputs.round_to_bf16(4 * rng.standard_normal((1, 4, 128)).astype(np.float32))     # large logits: sharp softmax
    k = inputs.round_to_bf16(rng.standard_normal((1, 2, 700, 128)).astype(np.float32))
    v = inputs.round_to_bf16(rng.standard_normal((1, 2, 700, 128)).astype(np.float32))
    for scale in (0.0, 0.5):
        for path in (F.PATH_AUTO, F.PATH_SIMT):
            assert np.allclose(_run(q, k, v, F.BF16, scale, path), O.decode_attention(q, k, v, scale), rtol=RTOL, atol=ATOL)


def test_over_the_compressed_cache_of_a_layer():
    """Compress a cfg3 layer, then attend over the compressed and over the full cache with a strided view."""
    wl = configs.get("cfg3")
    data = inputs.make_units(wl, [(20, 0)])
    p = oracle_params(wl, 1, 100)
    fp = F.Params(1, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, p.n_keep, dtype=F.BF16,
                  theta=wl.theta, tau=wl.tau_rel, tau_mode=F.TAU_REL)
    q, k, v = (to_dev(data[x], F.BF16) for x in "qkv")
    m = torch.from_numpy(data["modality"]).cuda()
    out = F.compress_layer_alloc(fp, q, k, v, m)
    q_dec = q[:, :, -1, :].contiguous()                              # the last window query stands in for the next token's
    for kk, vv in ((out["k_out"], out["v_out"]), (k, v)):
        o = torch.empty(q_dec.shape, dtype=torch.float32, device="cuda")
        ws = torch.empty(F.flowmm_decode_workspace_bytes(q_dec, kk, vv), dtype=torch.uint8, device="cuda")
        F.flowmm_decode_attention(q_dec, kk, vv, o, ws)
        ref = O.decode_attention(q_dec.float().cpu().numpy(), kk.float().cpu().numpy(), vv.float().cpu().numpy())
        assert np.allclose(o.cpu().numpy(), ref, rtol=RTOL, atol=ATOL)
    # strided K/V (a view into a larger buffer)
    big = torch.zeros((1, wl.n_kv_heads, wl.seq_len + 5, 2 * wl.head_dim), dtype=torch.bfloat16, device="cuda")
    kv = big[:, :, :wl.seq_len, :wl.head_dim]
    kv.copy_(k)
    o2 = torch.empty(q_dec.shape, dtype=torch.float32, device="cuda")
    ws = torch.empty(F.flowmm_decode_workspace_bytes(q_dec, kv, v), dtype=torch.uint8, device="cuda")
    F.flowmm_decode_attention(q_dec, kv, v, o2, ws)
    assert torch.equal(o2, o)


def test_decode_errors():
    q = torch.zeros((1, 18, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((1, 2, 64, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(F.FlowmmError) as e:                          # 9 query heads per KV head: not supported
        F.flowmm_decode_workspace_bytes(q, k, k)
    assert e.value.code == 2
    q = torch.zeros((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 4, 128), device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(F.FlowmmError) as e:
        F.flowmm_decode_attention(q, k, k, out, ws[:16])
    assert e.value.code == 5


@pytest.mark.parametrize("name,permille", [("cfg4", 1000), ("cfg4", 200), ("cfg2", 1000), ("cfg2", 100)])
def test_whole_stack_in_the_timed_configuration(name, permille):
    """Every layer of the stack as one call (what the bench times), full and compressed cache length;
    four layers are checked against the oracle."""
    wl = configs.get(name)
    q, k, v, _ = inputs.make_stack_device(wl, "cuda")
    n = wl.seq_len if permille == 1000 else wl.n_keep(permille)
    k, v = k[:, :, :n].contiguous(), v[:, :, :n].contiguous()
    q_dec = q[:, :, -1, :].contiguous()
    out = torch.full(q_dec.shape, float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(F.flowmm_decode_workspace_bytes(q_dec, k, v), dtype=torch.uint8, device="cuda")
    for _ in range(2):                                   # twice: the second call finds the scratch as the first left it
        F.flowmm_decode_attention(q_dec, k, v, out, ws)
        assert F.flowmm_last_device_status(ws) == 0
    assert torch.isfinite(out).all()
    for u in (0, wl.n_layers // 3, 2 * wl.n_layers // 3, wl.n_layers - 1):
        ref = O.decode_attention(q_dec[u:u + 1].float().cpu().numpy(), k[u:u + 1].float().cpu().numpy(),
                                 v[u:u + 1].float().cpu().numpy())
        got = out[u:u + 1].cpu().numpy()
        assert np.allclose(got, ref, rtol=RTOL, atol=ATOL), (u, np.abs(got - ref).max())
