"""flowmm_merge_static: the merge step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: inside another runtime's memory
pool, or as a plugin that is handed fixed buffers only.  For them the library carries a fixed
scratch array of its own and flowmm_merge_static uses that instead of a caller workspace.  This
file checks, through the C ABI, that the variant writes exactly what flowmm_merge writes, on two
calls in a row of different shape (the shared array still holds the first call's contents when
the second one starts), and that a problem too large for the array is refused before anything
is launched.  It is named to be collected last.
"""
import numpy as np
import pytest
import torch

from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import inputs

from gpu_util import gpu_params, to_dev

pytestmark = pytest.mark.gpu


def _case(seed, U, Hq, Hkv, D, L, W, B, **kw):
    """Random inputs, the pipeline's own decisions (through the existing entry points) and the
    existing merge's outputs for them."""
    rng = np.random.default_rng(seed)
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, **kw)
    fp = gpu_params(p, F.BF16)
    q = to_dev(inputs.round_to_bf16(rng.standard_normal((U, Hq, W, D)).astype(np.float32)), F.BF16)
    k = to_dev(inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32)), F.BF16)
    v = to_dev(inputs.round_to_bf16(rng.standard_normal((U, Hkv, L, D)).astype(np.float32)), F.BF16)
    m = torch.from_numpy((rng.random((U, L)) < 0.7).astype(np.uint8)).cuda()
    ref = F.compress_layer_alloc(fp, q, k, v, m)
    assert F.flowmm_last_device_status(ref["ws"]) == 0
    return fp, k, v, ref


def _run_static(fp, k, v, ref):
    k_out = torch.full_like(ref["k_out"], float("nan"))
    v_out = torch.full_like(ref["v_out"], float("nan"))
    F.flowmm_merge_static(fp, k, v, ref["retained"], ref["evicted"], ref["match"], ref["match_sim"], k_out, v_out)
    torch.cuda.synchronize()
    return k_out, v_out


def test_static_merge_equals_merge_on_two_calls_in_a_row():
    # long member lists (few pivots, intra-modal) so that the partial-sum scratch is used, then a
    # smaller problem of another shape that finds the array full of the first call's data
    first = _case(11, 2, 4, 2, 128, 900, 16, 5, flow_mode=O.FLOW_FORCE_INTRA)
    second = _case(12, 3, 2, 2, 128, 333, 8, 40, tau=3.0, tau_mode=O.TAU_REL)
    for fp, k, v, ref in (first, second, first):
        k_out, v_out = _run_static(fp, k, v, ref)
        # same kernels in the same fixed order: identical bits (the tests' K/V tolerance is
        # 2e-2 + 1e-2 |ref|; zero difference is inside it)
        assert torch.equal(k_out, ref["k_out"])
        assert torch.equal(v_out, ref["v_out"])


def test_static_merge_refuses_what_does_not_fit():
    fp = F.Params(64, 8, 8, 128, 40000, 16, 2000, dtype=F.BF16)      # needs far more than the 8 MiB array
    dummy = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(16, dtype=torch.int32, device="cuda")
    sim = torch.zeros(16, dtype=torch.float32, device="cuda")
    with pytest.raises(F.FlowmmError) as e:
        load = F.load()
        import ctypes
        cp = fp.c()
        code = load.flowmm_merge_static(ctypes.byref(cp), F._p(dummy), F._p(dummy), F._p(idx), F._p(idx), F._p(idx),
                                        F._p(sim), F._p(dummy), F._p(dummy), F._stream())
        F._check(code, "flowmm_merge_static")
    assert e.value.code == 5
    assert F.flowmm_last_launch_count() == 0
