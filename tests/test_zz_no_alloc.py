"""flowmm_merge_static: the merge step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: inside another runtime's memory
pool, or as a plugin that is handed fixed buffers only.  For them the library carries a fixed
scratch array of its own and flowmm_merge_static uses that instead of a caller workspace.  This
file checks, through the C ABI, that the variant writes exactly what flowmm_merge writes and what
the oracle's merge step gives, on calls in a row of different shapes that between them run every
merge kernel out of the shared array (which still holds the previous call's contents each time),
that a problem too large for the array is refused before anything is launched, and that the
status word inside the array can be read and cleared.  It is named to be collected last.
"""
import numpy as np
import pytest
import torch

from oracle import compare as C
from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import inputs

from gpu_util import gpu_params, to_dev

pytestmark = pytest.mark.gpu


def _case(seed, U, Hq, Hkv, D, L, W, B, dtype=F.BF16, path=F.PATH_AUTO, visual=0.7, admit=0, **kw):
    """Random inputs, the pipeline's own decisions (through the existing entry points), the existing
    merge's outputs for them and the oracle's merge of the same decisions.  admit > 0: tau is set
    between the admit-th and the next smallest pivot importance of the first head (from the oracle's
    scoring and selection), so that only about that many pivots may take non-pivots."""
    rng = np.random.default_rng(seed)
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, **kw)
    draw = lambda *shape: rng.standard_normal(shape).astype(np.float32)
    q, k, v = draw(U, Hq, W, D), draw(U, Hkv, L, D), draw(U, Hkv, L, D)
    if dtype == F.BF16:
        q, k, v = (inputs.round_to_bf16(x) for x in (q, k, v))
    m_np = (rng.random((U, L)) < visual).astype(np.uint8)
    if admit > 0:
        imp, _, _ = O.score(p, q, k, m_np)
        ret, _ = O.select(p, imp)
        piv = np.sort(imp[0, 0][ret[0, 0]])
        p.tau, p.tau_mode = float(0.5 * (piv[admit - 1] + piv[admit])), O.TAU_ABS
    fp = gpu_params(p, dtype, path)
    qd, kd, vd = (to_dev(x, dtype) for x in (q, k, v))
    m = torch.from_numpy(m_np).cuda()
    ref = F.compress_layer_alloc(fp, qd, kd, vd, m)
    assert F.flowmm_last_device_status(ref["ws"]) == 0
    ko, vo, _ = O.merge(p, k, v, ref["retained"].cpu().numpy(), ref["evicted"].cpu().numpy(),
                        ref["match"].cpu().numpy(), ref["match_sim"].cpu().numpy().astype(np.float64))
    return fp, kd, vd, ref, (ko, vo), dtype


def _run_static(fp, k, v, ref):
    k_out = torch.full_like(ref["k_out"], float("nan"))
    v_out = torch.full_like(ref["v_out"], float("nan"))
    F.flowmm_merge_static(fp, k, v, ref["retained"], ref["evicted"], ref["match"], ref["match_sim"], k_out, v_out)
    torch.cuda.synchronize()
    return k_out, v_out


def _check(case):
    fp, k, v, ref, oracle_kv, dtype = case
    k_out, v_out = _run_static(fp, k, v, ref)
    # same kernels in the same fixed order as flowmm_merge: identical bits
    assert torch.equal(k_out, ref["k_out"])
    assert torch.equal(v_out, ref["v_out"])
    # and the oracle's merge of the same decisions, at the tolerance of the parity tests
    for got, want in ((k_out, oracle_kv[0]), (v_out, oracle_kv[1])):
        got = got.float().cpu().numpy().astype(np.float64)
        if dtype == F.BF16:
            want = C.round_bf16(want)
            tol = 2e-2 + 1e-2 * np.abs(want)
        else:
            tol = 1e-4 + 1e-4 * np.abs(want)
        assert np.all(np.abs(got - want) <= tol)
    assert F.flowmm_merge_static_status() == 0


def test_static_merge_equals_merge_and_oracle_on_calls_in_a_row():
    # tensor-core merge (few slots): only the per-token table of the array is used
    few_slots = _case(11, 2, 4, 2, 128, 900, 16, 5, flow_mode=O.FLOW_FORCE_INTRA)
    small = _case(12, 3, 2, 2, 128, 333, 8, 40, tau=3.0, tau_mode=O.TAU_REL)
    # more than 240 slots: member lists sorted by slot, rows staged through shared memory; with a tau that admits
    # only eight of the 300 pivots the 2 700 non-pivots crowd into slots of several hundred members, which are cut
    # into pieces whose partial sums, arrival counters and work counter all live in the array
    long_lists = _case(13, 1, 2, 1, 128, 3000, 16, 300, visual=0.9, flow_mode=O.FLOW_FORCE_CROSS, admit=8)
    assert int(torch.bincount(long_lists[3]["match"][long_lists[3]["match"] >= 0].flatten()).max()) > 128
    # the register-gather merge: the SIMT path with five slots (pieces of 64 out of ~180 members per slot) ...
    simt = _case(14, 2, 2, 2, 128, 900, 16, 5, path=F.PATH_SIMT, flow_mode=O.FLOW_FORCE_CROSS)
    # ... and fp32 rows of 64 channels
    fp32 = _case(15, 2, 4, 2, 64, 700, 16, 6, dtype=F.F32, flow_mode=O.FLOW_FORCE_CROSS)
    # big -> small -> big, every kernel family finding the array full of another call's data
    for case in (long_lists, few_slots, simt, small, long_lists, fp32, simt, few_slots):
        _check(case)


def test_static_merge_status_word_is_read_and_cleared():
    assert F.flowmm_merge_static_status() == 0
    F.flowmm_merge_static_poke_status(8)                     # what a bounded wait that ran out would leave
    assert F.flowmm_merge_static_status() == 8
    assert F.flowmm_merge_static_status() == 0               # reading cleared it
    _check(_case(16, 1, 2, 2, 128, 400, 8, 20))              # and the array still serves a merge


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
