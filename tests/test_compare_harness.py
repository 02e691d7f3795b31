"""The comparison harness itself: it accepts the oracle's own (rounded) output and rejects
planted mistakes.  Mistakes are planted in copies of the oracle's output, on the CPU."""
import numpy as np
import pytest

from oracle import compare as C
from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import configs, inputs


def _case():
    wl = configs.get("cfg1")
    d = inputs.make_units(wl, [(0, 0)])
    p = O.OracleParams(1, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, wl.n_keep(250),
                       tau=wl.tau_rel, tau_mode=O.TAU_REL)
    out = O.compress_layer(p, d["q"], d["k"], d["v"], d["modality"])
    g = {key: out[key].copy() for key in ("importance", "rho", "strategy", "retained", "evicted", "match",
                                          "match_sim", "k_out", "v_out")}
    return p, d, g


def test_accepts_oracle_output():
    p, d, g = _case()
    stats = C.compare(p, d["q"], d["k"], d["v"], d["modality"], g, bf16_out=False)
    assert stats["k_out_max_abs"] == 0 and stats["match_near_ties"] == 0


def test_round_bf16_matches_bit_rounding():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(10000).astype(np.float32)
    assert np.array_equal(C.round_bf16(x.astype(np.float64)), inputs.round_to_bf16(x).astype(np.float64))
    assert C.round_bf16(np.array([1.0 + 2 ** -8]))[0] == 1.0 and C.round_bf16(np.array([1.0 + 3 * 2 ** -8]))[0] == 1.0 + 2 ** -6


@pytest.mark.parametrize("mistake", ["importance", "swap_pivot", "match", "sim", "k_out", "rho", "not_ascending"])
def test_rejects_planted_mistakes(mistake):
    p, d, g = _case()
    if mistake == "importance":
        g["importance"][0, 1, 50] *= 1.01
    elif mistake == "swap_pivot":
        r, e = g["retained"][0, 0].copy(), g["evicted"][0, 0].copy()
        imp = g["importance"][0, 0]
        worst_e = int(np.argmin(imp[e]))
        r[0], e[worst_e] = e[worst_e], r[0]
        g["retained"][0, 0], g["evicted"][0, 0] = np.sort(r), np.sort(e)
    elif mistake == "match":
        j = int(np.nonzero(g["match"][0, 2] >= 0)[0][0])
        g["match"][0, 2, j] = (g["match"][0, 2, j] + 1) % p.n_keep
    elif mistake == "sim":
        j = int(np.nonzero(g["match"][0, 2] >= 0)[0][0])
        g["match_sim"][0, 2, j] += 0.01
    elif mistake == "k_out":
        g["k_out"][0, 3, 5, 7] += 0.05
    elif mistake == "rho":
        g["rho"][0] *= 1.01
    elif mistake == "not_ascending":
        g["retained"][0, 0, :2] = g["retained"][0, 0, :2][::-1]
    with pytest.raises(C.ParityError):
        C.compare(p, d["q"], d["k"], d["v"], d["modality"], g, bf16_out=False)


def test_sampled_rows_judge_only_what_the_oracle_matched():
    """With a row sample the harness still rejects a wrong match inside the sample, and a slot that received a
    non-pivot outside the sample is left out of the K/V comparison instead of being judged on the other side's
    own match."""
    p, d, g = _case()
    E = p.seq_len - p.n_keep
    sel = np.random.default_rng(3).random((1, p.n_kv_heads, E)) < 0.5     # the sample compare() draws for seed 3
    stats = C.compare(p, d["q"], d["k"], d["v"], d["modality"], g, bf16_out=False, row_fraction=0.5, row_seed=3)
    assert stats["match_rows_checked"] == int(sel.sum()) < stats["match_rows_total"]
    assert stats["kv_rows_checked"] < stats["kv_rows_total"]
    # a wrong match outside the sample, with K/V that follow it: not judged (and not accepted as checked either)
    h = 2
    outside = [j for j in np.nonzero(~sel[0, h])[0] if g["match"][0, h, j] >= 0]
    inside = [j for j in np.nonzero(sel[0, h])[0] if g["match"][0, h, j] >= 0]
    bad = {key: val.copy() for key, val in g.items()}
    j = outside[0]
    bad["match"][0, h, j] = (bad["match"][0, h, j] + 1) % p.n_keep
    forced = O.merge(p, d["k"], d["v"], bad["retained"], bad["evicted"], bad["match"], bad["match_sim"])
    bad["k_out"], bad["v_out"] = forced[0], forced[1]
    C.compare(p, d["q"], d["k"], d["v"], d["modality"], bad, bf16_out=False, row_fraction=0.5, row_seed=3)
    with pytest.raises(C.ParityError):                                     # the full check does see it
        C.compare(p, d["q"], d["k"], d["v"], d["modality"], bad, bf16_out=False)
    # the same mistake inside the sample is rejected
    bad = {key: val.copy() for key, val in g.items()}
    j = inside[0]
    bad["match"][0, h, j] = (bad["match"][0, h, j] + 1) % p.n_keep
    with pytest.raises(C.ParityError):
        C.compare(p, d["q"], d["k"], d["v"], d["modality"], bad, bf16_out=False, row_fraction=0.5, row_seed=3)
