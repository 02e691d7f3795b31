"""The workloads at their full sizes, in the launch shape the benchmark times (a whole stack of
units in one flowmm_compress_layer call), against the oracle on sampled units (every token and
every non-pivot row of those units); structural invariants on every unit."""
import numpy as np
import pytest
import torch

from oracle import compare as C
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

from gpu_util import oracle_params, run_gpu

pytestmark = pytest.mark.gpu


def _unit_slice(g, idx):
    return {key: np.ascontiguousarray(val[idx]) for key, val in g.items()}


def _stack_check(name, units, permille, sample):
    wl = configs.get(name)
    data = inputs.make_units(wl, units)
    p_all = oracle_params(wl, len(units), permille)
    g = run_gpu(p_all, data["q"], data["k"], data["v"], data["modality"], F.BF16)
    C.check_structure(p_all, g, data["modality"])                # every unit
    idx = np.asarray(sample)
    p = oracle_params(wl, len(sample), permille)
    stats = C.compare(p, data["q"][idx], data["k"][idx], data["v"][idx], data["modality"][idx], _unit_slice(g, idx),
                      bf16_out=True)
    assert stats["match_rows_checked"] == stats["match_rows_total"] and stats["kv_rows_checked"] == stats["kv_rows_total"]
    # both merging strategies must occur in a whole stack (the generator is tuned for that)
    if len(units) >= 20:
        assert 0 < int(g["strategy"].sum()) < len(units)
    return stats


def test_cfg2_whole_stack():
    wl = configs.get("cfg2")
    _stack_check("cfg2", [(l, 0) for l in range(wl.n_layers)], 100, [0, 9, 16, 31])


def test_cfg3_whole_stack():
    wl = configs.get("cfg3")
    _stack_check("cfg3", [(l, 0) for l in range(wl.n_layers)], 100, [0, 13, 27])


@pytest.mark.parametrize("permille", [50, 200])
def test_cfg4_whole_stack(permille):
    wl = configs.get("cfg4")
    _stack_check("cfg4", [(l, 0) for l in range(wl.n_layers)], permille, [5, 22])


def test_cfg5_long_context_units():
    # two (layer, sequence) units of the long-context workload in one call, the first of an intra-modal and
    # the second of a cross-modal layer; the oracle scores every token and matches every non-pivot
    stats = _stack_check("cfg5", [(0, 0), (79, 3)], 50, [0, 1])
    assert stats["match_rows_total"] == 2 * 8 * (33792 - 1690)


def test_cfg5_whole_stack_as_benchmarked():
    """The benchmark's own launch: all 80 layers x 4 sequences (320 units, 44 GB of K and V) in one call,
    inputs drawn on the device as the benchmark draws them.  Structural invariants on every unit; two units
    (an early intra-modal layer, a late cross-modal one) are copied out and compared with the oracle in full."""
    wl = configs.get("cfg5")
    q, k, v, m = inputs.make_stack_device(wl, "cuda")
    U = q.shape[0]
    assert U == 320
    fp = F.Params(U, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, wl.n_keep(50), dtype=F.BF16,
                  theta=wl.theta, tau=wl.tau_rel, tau_mode=F.TAU_REL)
    out = F.compress_layer_alloc(fp, q, k, v, m)
    assert F.flowmm_last_device_status(out["ws"]) == 0
    g = {key: (t.float().cpu().numpy() if t.is_floating_point() and key not in ("k_out", "v_out") else t)
         for key, t in out.items() if key != "ws"}
    structure = {key: (val if isinstance(val, np.ndarray) else val.cpu().numpy()) for key, val in g.items()
                 if key not in ("k_out", "v_out")}
    structure["importance"] = structure["importance"].astype(np.float64)
    structure["rho"] = structure["rho"].astype(np.float64)
    mod_np = m.cpu().numpy()
    C.check_structure(oracle_params(wl, U, 50), structure, mod_np)
    assert 0 < int(structure["strategy"].sum()) < U                    # both merging strategies occur
    strat = structure["strategy"]
    intra_u = int(np.nonzero(strat == 0)[0][1])                        # layer 0, sequence 1
    cross_u = int(np.nonzero(strat == 1)[0][-2])                       # last layer, sequence 2
    for u in (intra_u, cross_u):
        gu = {key: np.ascontiguousarray(val[u:u + 1]) for key, val in structure.items()}
        gu["match_sim"] = gu["match_sim"].astype(np.float64)
        for key in ("k_out", "v_out"):
            gu[key] = out[key][u:u + 1].float().cpu().numpy().astype(np.float64)
        stats = C.compare(oracle_params(wl, 1, 50), q[u:u + 1].float().cpu().numpy(), k[u:u + 1].float().cpu().numpy(),
                          v[u:u + 1].float().cpu().numpy(), mod_np[u:u + 1], gu, bf16_out=True)
        assert stats["match_rows_checked"] == stats["match_rows_total"]
    del out, q, k, v
    torch.cuda.empty_cache()
