"""CUDA path against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from oracle import compare as C
from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

from gpu_util import oracle_params, run_gpu

pytestmark = pytest.mark.gpu


def _dtype(wl):
    return F.BF16 if wl.dtype == "bf16" else F.F32


def _check(wl, units, permille, path=F.PATH_AUTO, **kw):
    data = inputs.make_units(wl, units)
    p = oracle_params(wl, len(units), permille, **kw)
    g = run_gpu(p, data["q"], data["k"], data["v"], data["modality"], _dtype(wl), path)
    return C.compare(p, data["q"], data["k"], data["v"], data["modality"], g, bf16_out=wl.dtype == "bf16")


def test_cfg1_fp32():
    stats = _check(configs.get("cfg1"), [(0, 0)], 250)
    assert stats["k_out_max_abs"] < 1e-4


@pytest.mark.parametrize("path", [F.PATH_AUTO, F.PATH_SIMT])
@pytest.mark.parametrize("permille", [50, 100, 200])
def test_cfg2_sampled_layers(permille, path):
    # layers on both sides of the theta crossing, several units in one call
    _check(configs.get("cfg2"), [(0, 0), (15, 0), (16, 0), (31, 0)], permille, path)


@pytest.mark.parametrize("path", [F.PATH_AUTO, F.PATH_SIMT])
def test_cfg3_gqa(path):
    _check(configs.get("cfg3"), [(0, 0), (13, 0), (27, 0)], 100, path)


@pytest.mark.parametrize("permille", [50, 200])
def test_cfg4_video_mixed_window(permille):
    _check(configs.get("cfg4"), [(2, 0), (20, 0)], permille)


@pytest.mark.parametrize("mode", ["mean", "force_intra", "force_cross", "misaligned", "no_flow_no_gate", "no_gate",
                                  "keep_window", "abs_tau"])
def test_variants(mode):
    wl = configs.get("cfg2")
    kw = {"mean": dict(merge_mode=O.MERGE_MEAN), "force_intra": dict(flow_mode=O.FLOW_FORCE_INTRA),
          "force_cross": dict(flow_mode=O.FLOW_FORCE_CROSS), "misaligned": dict(flow_mode=O.FLOW_MISALIGNED),
          "no_flow_no_gate": dict(flow_mode=O.FLOW_FORCE_CROSS, tau=float("inf")), "no_gate": dict(tau=float("inf")),
          "keep_window": dict(keep_window=1), "abs_tau": dict(tau=0.3, tau_mode=O.TAU_ABS)}[mode]
    _check(wl, [(3, 0), (29, 0)], 100, **kw)


def _random_case(rng, U, Hq, Hkv, D, L, W, B, dtype, vis_frac=0.6, **kw):
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, **kw)
    q = rng.standard_normal((U, Hq, W, D)).astype(np.float32)
    k = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
    v = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
    m = (rng.random((U, L)) < vis_frac).astype(np.uint8)
    if dtype == F.BF16:
        q, k, v = inputs.round_to_bf16(q), inputs.round_to_bf16(k), inputs.round_to_bf16(v)
    g = run_gpu(p, q, k, v, m, dtype)
    return C.compare(p, q, k, v, m, g, bf16_out=dtype == F.BF16)


@pytest.mark.parametrize("dtype", [F.F32, F.BF16])
@pytest.mark.parametrize("D", [64, 128])
def test_ragged_shapes(dtype, D):
    rng = np.random.default_rng(100 + D + dtype)
    # sizes that are multiples of no tile: several tiles plus a ragged tail in every dimension
    for (U, Hq, Hkv, L, W, B) in [(2, 6, 2, 333, 21, 37), (1, 3, 3, 1031, 5, 300), (3, 4, 1, 130, 64, 129)]:
        _random_case(rng, U, Hq, Hkv, D, L, W, B, dtype, tau=3.0, tau_mode=O.TAU_REL, theta=0.5)


def test_member_lists_too_long_for_the_shared_memory_sort():
    # 35 700 non-pivots per head: six bytes each no longer fit the sort's shared-memory staging, so the member lists of the
    # staged merge are sorted through global memory (the shorter lists of every other case take the staged sort)
    rng = np.random.default_rng(4242)
    stats = _random_case(rng, 1, 2, 1, 128, 36000, 16, 300, F.BF16, vis_frac=0.8, tau=3.0, tau_mode=O.TAU_REL, theta=0.5)
    assert stats["kv_rows_checked"] == stats["kv_rows_total"]


def test_short_context_kernel_boundaries():
    """Shapes around the switch points of the one-pass scoring kernel (32 proxy rows per KV head, up to 8 key
    tiles), the short-list matching kernel (up to 256 candidate columns, i.e. B <= 224) and the tensor-core merge
    (B <= 240), with ragged lengths and windows that straddle a tile edge."""
    rng = np.random.default_rng(23)
    for (U, Hq, Hkv, L, W, B) in [
        (2, 2, 2, 333, 32, 40),      # G W = 32, three key tiles, ragged tail
        (1, 4, 2, 1000, 16, 96),     # G = 2, W = 16, eight key tiles; 96 pivots: 128 candidate columns
        (2, 1, 1, 129, 32, 1),       # window across the tile edge, a single pivot
        (1, 2, 2, 1024, 32, 224),    # the longest context of the one-pass kernel; 256 candidate columns
        (1, 2, 2, 1025, 32, 225),    # one token and one pivot more: two-pass scoring, general matching kernel
        (1, 2, 1, 600, 32, 240),     # the largest budget of the tensor-core merge
        (1, 2, 1, 600, 32, 241),     # one more: gather merge
        (3, 2, 2, 64, 32, 33),       # half of the prompt is the window
    ]:
        _random_case(rng, U, Hq, Hkv, 128, L, W, B, F.BF16, tau=3.0, tau_mode=O.TAU_REL, theta=0.5)
    # every layer forced either way, and pivots all protected (nothing is merged: the compaction alone)
    _random_case(rng, 2, 2, 2, 128, 640, 32, 64, F.BF16, flow_mode=O.FLOW_FORCE_INTRA, vis_frac=0.8)
    _random_case(rng, 2, 2, 2, 128, 640, 32, 64, F.BF16, flow_mode=O.FLOW_FORCE_CROSS, merge_mode=O.MERGE_MEAN)
    _random_case(rng, 1, 2, 2, 128, 640, 32, 64, F.BF16, tau=0.0)
    _random_case(rng, 1, 2, 2, 128, 300, 32, 100, F.BF16, keep_window=1, tau=float("inf"))


def test_degenerate_cases():
    rng = np.random.default_rng(7)
    _random_case(rng, 1, 2, 2, 64, 50, 50, 1, F.F32)                       # one pivot, window = whole prompt
    _random_case(rng, 1, 2, 2, 64, 77, 3, 77, F.BF16)                      # full budget: identity
    _random_case(rng, 2, 2, 1, 128, 96, 8, 20, F.BF16, vis_frac=0.0)       # text only: rho = 0
    _random_case(rng, 2, 2, 1, 128, 96, 8, 20, F.BF16, vis_frac=1.0)       # visual only
    _random_case(rng, 1, 4, 2, 64, 90, 4, 9, F.F32, tau=0.0)               # every pivot protected: pure eviction
    _random_case(rng, 1, 1, 1, 64, 1, 1, 1, F.F32)                         # a single token
    _random_case(rng, 1, 2, 2, 128, 700, 16, 3, F.BF16, flow_mode=O.FLOW_FORCE_INTRA, vis_frac=0.9)   # long member lists


def test_full_budget_is_bit_exact_copy():
    wl = configs.get("cfg2")
    data = inputs.make_units(wl, [(5, 0)])
    p = oracle_params(wl, 1, 1000)
    g = run_gpu(p, data["q"], data["k"], data["v"], data["modality"], F.BF16)
    assert np.array_equal(g["k_out"], data["k"].astype(np.float64))
    assert np.array_equal(g["v_out"], data["v"].astype(np.float64))


def test_duplicate_keys_and_run_to_run_determinism():
    rng = np.random.default_rng(3)
    wl = configs.get("cfg2")
    data = inputs.make_units(wl, [(20, 0)])
    k = data["k"].copy()
    k[0, :, 100] = k[0, :, 400]            # two identical visual keys in every head
    p = oracle_params(wl, 1, 100)
    a = run_gpu(p, data["q"], k, data["v"], data["modality"], F.BF16)
    b = run_gpu(p, data["q"], k, data["v"], data["modality"], F.BF16)
    for key in a:
        assert np.array_equal(a[key], b[key]), key
    C.compare(p, data["q"], k, data["v"], data["modality"], a, bf16_out=True)
    # whenever exactly one of the twins is a pivot, the other matches it with similarity 1
    for h in range(wl.n_kv_heads):
        ret, evi = a["retained"][0, h], a["evicted"][0, h]
        for piv, other in ((100, 400), (400, 100)):
            if piv in ret and other in evi:
                j = int(np.nonzero(evi == other)[0][0])
                slot = int(np.nonzero(ret == piv)[0][0])
                if a["match"][0, h, j] >= 0 and a["importance"][0, h, piv] <= wl.tau_rel * wl.window / wl.seq_len:
                    assert a["match"][0, h, j] == slot and abs(a["match_sim"][0, h, j] - 1) < 1e-5


def test_strided_inputs():
    """K/V/Q taken as views of larger buffers (padding between tokens and heads)."""
    import torch
    rng = np.random.default_rng(17)
    U, Hq, Hkv, D, L, W, B = 2, 4, 2, 128, 200, 8, 30
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, tau=5.0, tau_mode=O.TAU_REL)
    q = inputs.round_to_bf16(rng.standard_normal((U, Hq, W, D)).astype(np.float32))
    k = inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32))
    v = inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32))
    m = (rng.random((U, L)) < 0.5).astype(np.uint8)
    fp = F.Params(U, Hq, Hkv, D, L, W, B, dtype=F.BF16, tau=5.0, tau_mode=F.TAU_REL)
    big_k = torch.zeros((U, Hkv, L + 3, D + 8), dtype=torch.bfloat16, device="cuda")
    big_v = torch.zeros((U, Hkv + 1, L, D + 16), dtype=torch.bfloat16, device="cuda")
    big_q = torch.zeros((U, Hq, W, 2 * D), dtype=torch.bfloat16, device="cuda")
    kd, vd, qd = big_k[:, :, :L, :D], big_v[:, :Hkv, :, :D], big_q[:, :, :, :D]
    kd.copy_(torch.from_numpy(k)); vd.copy_(torch.from_numpy(v)); qd.copy_(torch.from_numpy(q))
    out = F.compress_layer_alloc(fp, qd, kd, vd, torch.from_numpy(m).cuda())
    g = {key: (t.float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy())
         for key, t in out.items() if key != "ws"}
    C.compare(p, q, k, v, m, g, bf16_out=True)
