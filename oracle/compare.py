"""Compares outputs of the CUDA path with the fp64 oracle (TEST INFRASTRUCTURE).

Takes plain numpy arrays from both sides; imports nothing from the CUDA package.
Tolerances (stated once, here):
  * importance, rho, match_sim: relative 1e-3 (plus an absolute floor far below
    any value that can influence a decision);
  * index sets, strategy, match: identical, except where the oracle's own margin
    at that decision is below 1e-4 relative (top-B boundary, best vs runner-up
    similarity, importance vs tau, rho vs theta); such a decision may go either
    way, and the oracle's later steps are then re-run with the other side's
    decision forced before K/V are compared;
  * merged K/V: |x - ref| <= 2e-2 + 1e-2 |ref| for bf16 outputs against the bf16
    rounding of the oracle's fp64 result; 1e-4 + 1e-4 |ref| for fp32 outputs.
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from . import flowmm_oracle as O

SCORE_RTOL = 1e-3
GAP_RTOL = 1e-4
IMPORTANCE_ATOL = 1e-30
SIM_ATOL = 1e-6


def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bf16 (ties to even), returned as float64.  Via float32 first would
    double-round, so round the float64 directly on its float32-exponent grid."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = x != 0
    e = np.floor(np.log2(np.abs(x[nz])))
    ulp = np.exp2(e - 7)                       # bf16 keeps 8 significant bits
    out[nz] = np.rint(x[nz] / ulp) * ulp       # rint is ties-to-even
    return out


class ParityError(AssertionError):
    pass


def _require(cond, msg):
    if not cond:
        raise ParityError(msg)


def check_structure(p: O.OracleParams, g: Dict[str, np.ndarray], modality: np.ndarray):
    """Properties that hold for any correct output, at any size, without the oracle."""
    L, B, W = p.seq_len, p.n_keep, p.window
    imp = g["importance"]
    _require(np.all(np.isfinite(imp)) and np.all(imp >= 0), "importance must be finite and non-negative")
    _require(np.allclose(imp.sum(-1), W, rtol=1e-3), "importance of a head must sum to W")
    _require(np.all((g["rho"] >= 0) & (g["rho"] <= 1 + 1e-6)), "rho outside [0, 1]")
    ret, evi = g["retained"], g["evicted"]
    _require(ret.shape[-1] == B and evi.shape[-1] == L - B, "budget: exactly B pivots per head")
    both = np.sort(np.concatenate([ret, evi], axis=-1), axis=-1)
    _require(np.array_equal(both, np.broadcast_to(np.arange(L, dtype=both.dtype), both.shape)),
             "pivots and non-pivots must partition the tokens")
    _require(np.all(np.diff(ret, axis=-1) > 0) and (L - B < 2 or np.all(np.diff(evi, axis=-1) > 0)),
             "index lists must ascend")
    if L > B:
        piv_imp = np.take_along_axis(imp, ret.astype(np.int64), -1)
        if p.keep_window:                      # forced window pivots are exempt from the ranking
            piv_imp = np.where(ret >= L - W, np.inf, piv_imp)
            _require(np.all((ret >= L - W).sum(-1) == W), "keep_window: a proxy token was evicted")
        hi = np.take_along_axis(imp, evi.astype(np.int64), -1).max(-1)
        _require(np.all(piv_imp.min(-1) >= hi), "a non-pivot outranks a pivot")
        mt = g["match"]
        _require(np.all((mt >= -1) & (mt < B)), "match out of range")
        _require(np.all(np.abs(g["match_sim"]) <= 1 + 1e-5), "cosine outside [-1, 1]")
        _require(np.all(g["match_sim"][mt < 0] == 0), "unmatched rows carry similarity 0")
        intra = g["strategy"] == O.INTRA
        for u in np.nonzero(intra)[0]:
            hit = mt[u] >= 0
            piv = np.take_along_axis(ret[u], np.where(hit, mt[u], 0).astype(np.int64), -1)
            _require(np.all((modality[u][piv] == modality[u][evi[u]]) | ~hit), "intra-modal layer merged across modalities")


def compare(p: O.OracleParams, q, k, v, modality, g: Dict[str, np.ndarray], bf16_out: bool,
            row_fraction: float = 1.0, row_seed: int = 0) -> Dict[str, float]:
    """Raises ParityError on the first violation; returns a few statistics otherwise.
    `g` holds the CUDA path's importance, rho, strategy, retained, evicted, match, match_sim,
    k_out, v_out as numpy arrays (k_out / v_out as float32 or float64 values).

    row_fraction < 1: the oracle matches only a seeded random sample of the non-pivots (every one
    with that probability).  Output rows that received a non-pivot outside the sample cannot be
    judged by the oracle (their merge would rest on the other side's own match) and are left out
    of the K/V comparison; the statistics say how many rows were matched by the oracle
    (`match_rows_checked`, `match_rows_total`) and how many output rows were compared
    (`kv_rows_checked`, `kv_rows_total`)."""
    stats: Dict[str, float] = {}
    check_structure(p, g, modality)
    U, Hkv, L, B = p.n_units, p.n_kv_heads, p.seq_len, p.n_keep
    E = L - B
    imp, cross, total = O.score(p, q, k, modality)
    err = np.abs(g["importance"] - imp)
    _require(np.all(err <= SCORE_RTOL * np.abs(imp) + IMPORTANCE_ATOL),
             "importance off by rel %.3g" % np.max(err / (np.abs(imp) + IMPORTANCE_ATOL)))
    stats["importance_max_rel"] = float(np.max(err / (np.abs(imp) + 1e-300)))
    rho, strat = O.layer_flow(p, cross, total)
    _require(np.allclose(g["rho"], rho, rtol=SCORE_RTOL, atol=1e-7), "rho differs")
    flip = g["strategy"] != strat
    if p.flow_mode == O.FLOW_AUTO and p.theta > 0:
        _require(np.all(np.abs(rho[flip] - p.theta) <= GAP_RTOL * p.theta), "strategy differs away from theta")
    else:
        _require(not flip.any(), "strategy differs")
    stats["strategy_near_ties"] = int(flip.sum())

    ret, evi = O.select(p, imp)
    n_set_ties = 0
    for u in range(U):
        for h in range(Hkv):
            if np.array_equal(ret[u, h], g["retained"][u, h]):
                continue
            diff = np.setxor1d(ret[u, h], g["retained"][u, h])
            if p.keep_window:                  # the boundary among the tokens that compete for a place
                free = imp[u, h][: L - p.window]
                bound = np.sort(free)[::-1][B - p.window - 1] if B > p.window else np.inf
            else:
                bound = np.sort(imp[u, h])[::-1][B - 1]
            _require(np.all(np.abs(imp[u, h][diff] - bound) <= GAP_RTOL * bound),
                     "pivot set differs away from the top-B boundary (unit %d head %d)" % (u, h))
            n_set_ties += len(diff) // 2
    stats["select_near_ties"] = n_set_ties

    # from here on follow the CUDA path's (validated) decisions
    forced = {"strategy": g["strategy"], "retained": g["retained"], "evicted": g["evicted"]}
    row_select = None
    if row_fraction < 1.0 and E > 0:
        row_select = np.random.default_rng(row_seed).random((U, Hkv, E)) < row_fraction
    mt, sim, ru = O.match(p, k, imp, modality, forced["retained"], forced["evicted"], forced["strategy"], row_select)
    tau_eff = p.tau * p.window / p.seq_len if p.tau_mode == O.TAU_REL else p.tau
    n_match_ties = 0
    sim_forced = sim.copy()
    if E > 0:
        evaluated = mt != -2
        bad = evaluated & (mt != g["match"])
        for u, h, j in zip(*np.nonzero(bad)):
            e = forced["evicted"][u, h, j]
            gs, os_ = g["match"][u, h, j], mt[u, h, j]

            def near_gate(slot):
                i_piv = imp[u, h, forced["retained"][u, h, slot]]
                return np.isfinite(tau_eff) and abs(i_piv - tau_eff) <= GAP_RTOL * abs(tau_eff)

            ok = False
            if gs >= 0:
                r = forced["retained"][u, h, gs]
                admissible = (imp[u, h, r] <= tau_eff or near_gate(gs)) and \
                    (forced["strategy"][u] == O.CROSS or modality[u, r] == modality[u, e])
                ug = O.cosine(k[u, h, e], k[u, h, r])
                sim_forced[u, h, j] = ug
                if admissible:
                    ok = os_ < 0 and near_gate(gs) or (os_ >= 0 and (
                        abs(ug - sim[u, h, j]) <= GAP_RTOL * abs(sim[u, h, j]) or near_gate(os_)))
            else:
                sim_forced[u, h, j] = 0.0
                ok = os_ >= 0 and near_gate(os_)
            _require(ok, "match differs away from a tie (unit %d head %d row %d: %d vs oracle %d)" % (u, h, j, gs, os_))
            n_match_ties += 1
        same = evaluated & ~bad
        serr = np.abs(g["match_sim"] - sim)[same]
        _require(np.all(serr <= SCORE_RTOL * np.abs(sim[same]) + SIM_ATOL), "match_sim off by %.3g" % serr.max(initial=0))
        stats["match_sim_max_abs"] = float(serr.max(initial=0))
    stats["match_near_ties"] = n_match_ties
    # Output rows the oracle can judge: those whose every member (non-pivot matched to the slot by the
    # other side) was matched by the oracle too.  With the full check that is every row.
    row_ok = np.ones((U, Hkv, B), dtype=bool)
    if E > 0:
        unchecked = ~evaluated & (g["match"] >= 0)
        for u, h, j in zip(*np.nonzero(unchecked)):
            row_ok[u, h, g["match"][u, h, j]] = False
        stats["match_rows_checked"] = int(evaluated.sum())
        stats["match_rows_total"] = int(evaluated.size)
        sim_forced = np.where(evaluated, sim_forced, g["match_sim"])      # only feeds rows that are left out below
    stats["kv_rows_checked"] = int(row_ok.sum())
    stats["kv_rows_total"] = int(row_ok.size)

    ko, vo, _ = O.merge(p, k, v, forced["retained"], forced["evicted"], g["match"], sim_forced)
    for name, ref in (("k_out", ko), ("v_out", vo)):
        got = np.asarray(g[name], dtype=np.float64)
        if bf16_out:
            ref = round_bf16(ref)
            tol = 2e-2 + 1e-2 * np.abs(ref)
        else:
            tol = 1e-4 + 1e-4 * np.abs(ref)
        d = np.abs(got - ref)[row_ok]
        _require(np.all(d <= tol[row_ok]), "%s off: max abs err %.4g" % (name, d.max(initial=0)))
        stats[name + "_max_abs"] = float(d.max(initial=0))
        stats[name + "_exact_frac"] = float(np.mean(d == 0)) if d.size else 1.0
    return stats
