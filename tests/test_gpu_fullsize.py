"""The workloads at their full sizes, in the launch shape the benchmark times (a whole stack of
units in one flowmm_compress_layer call), against the oracle on sampled units; structural
invariants on every unit."""
import numpy as np
import pytest

from oracle import compare as C
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

from gpu_util import oracle_params, run_gpu

pytestmark = pytest.mark.gpu


def _unit_slice(g, idx):
    return {key: np.ascontiguousarray(val[idx]) for key, val in g.items()}


def _stack_check(name, units, permille, sample, row_step=1):
    wl = configs.get(name)
    data = inputs.make_units(wl, units)
    p_all = oracle_params(wl, len(units), permille)
    g = run_gpu(p_all, data["q"], data["k"], data["v"], data["modality"], F.BF16)
    C.check_structure(p_all, g, data["modality"])                # every unit
    idx = np.asarray(sample)
    p = oracle_params(wl, len(sample), permille)
    stats = C.compare(p, data["q"][idx], data["k"][idx], data["v"][idx], data["modality"][idx], _unit_slice(g, idx),
                      bf16_out=True, row_step=row_step)
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
    _stack_check("cfg4", [(l, 0) for l in range(wl.n_layers)], permille, [5, 22], row_step=4)


def test_cfg5_long_context_units():
    # two (layer, sequence) units of the long-context workload in one call; the oracle scores every
    # token and matches every 32nd non-pivot
    _stack_check("cfg5", [(0, 0), (79, 3)], 50, [0, 1], row_step=32)
