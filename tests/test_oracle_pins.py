"""Pins for the fp64 oracle: closed forms, invariants, library routines, brute force.

None of these call the oracle to make their own expectation: each expected
value comes from exact rational arithmetic, a hand-worked fixture, a numpy /
scipy / scikit-learn routine, or enumeration of every candidate on tiny inputs.
"""
import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy.cluster.vq import vq
from scipy.special import softmax
from sklearn.metrics.pairwise import cosine_similarity

from oracle import flowmm_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))


def params(U=1, Hq=2, Hkv=2, D=4, L=10, W=3, B=4, **kw):
    return O.OracleParams(U, Hq, Hkv, D, L, W, B, **kw)


def rand_unit(rng, p, vis_frac=0.5):
    q = rng.standard_normal((p.n_units, p.n_q_heads, p.window, p.head_dim)).astype(np.float32)
    k = rng.standard_normal((p.n_units, p.n_kv_heads, p.seq_len, p.head_dim)).astype(np.float32)
    v = rng.standard_normal((p.n_units, p.n_kv_heads, p.seq_len, p.head_dim)).astype(np.float32)
    m = (rng.random((p.n_units, p.seq_len)) < vis_frac).astype(np.uint8)
    return q, k, v, m


# ---------------------------------------------------------------- score / flow

def test_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "hand_worked_eq8.json")))
    p = params(Hq=1, Hkv=1, D=1, L=3, W=2, B=1, softmax_scale=1.0)
    k = np.array(g["keys"], dtype=np.float32).reshape(1, 1, 3, 1)
    q = np.array(g["queries"], dtype=np.float32).reshape(1, 1, 2, 1)
    m = np.array(g["modality"], dtype=np.uint8).reshape(1, 3)
    imp, cross, total = O.score(p, q, k, m)
    np.testing.assert_allclose(imp[0, 0], g["importance"], rtol=0, atol=2e-7)   # ln 2, ln 3 are float32 inputs
    assert abs(cross[0, 0] - g["cross_mass"]) < 2e-7
    assert abs(total[0, 0] - g["total_mass"]) < 1e-12
    rho, _ = O.layer_flow(p, cross, total)
    assert abs(rho[0] - g["rho"]) < 2e-7
    ret, evi = O.select(p, imp)
    assert ret[0, 0].tolist() == g["top1_retained"]
    assert evi[0, 0].tolist() == [0, 2]


@pytest.mark.parametrize("G", [1, 3])
def test_zero_queries_closed_form(G):
    """Q = 0 makes every causal row uniform: alpha[a, i] = 1 / (p_a + 1) for i <= p_a."""
    rng = np.random.default_rng(5)
    L, W, Hkv = 23, 7, 2
    p = params(Hq=Hkv * G, Hkv=Hkv, D=8, L=L, W=W, B=5)
    q, k, v, m = rand_unit(rng, p)
    q[:] = 0
    imp, cross, total = O.score(p, q, k, m)
    exp_imp = [sum(Fraction(1, L - W + a + 1) for a in range(W) if L - W + a >= i) for i in range(L)]
    exp_cross = sum(Fraction(sum(1 for i in range(L - W + a + 1) if m[0, i] != m[0, L - W + a]), L - W + a + 1)
                    for a in range(W))
    for h in range(Hkv):
        np.testing.assert_allclose(imp[0, h], [float(x) for x in exp_imp], rtol=1e-13)
    np.testing.assert_allclose(cross[0], float(exp_cross), rtol=1e-13)
    np.testing.assert_allclose(total[0], W, rtol=1e-13)
    rho, _ = O.layer_flow(p, cross, total)
    assert abs(rho[0] - float(exp_cross / W)) < 1e-13


@pytest.mark.parametrize("G", [1, 2])
def test_score_equals_library_softmax(G):
    """Eq. 8 through scipy's softmax and numpy's matmul, on the small fp32 workload's shape."""
    rng = np.random.default_rng(11)
    Hkv, D, L, W = 4 // G, 64, 192, 16
    p = params(Hq=4, Hkv=Hkv, D=D, L=L, W=W, B=48)
    q, k, v, m = rand_unit(rng, p, vis_frac=0.7)
    imp, cross, total = O.score(p, q, k, m)
    pos = L - W + np.arange(W)
    mask = np.where(np.arange(L)[None, :] <= pos[:, None], 0.0, -np.inf)
    exp_imp = np.zeros((Hkv, L))
    for g in range(4):
        h = g // G
        logits = q[0, g].astype(np.float64) @ k[0, h].astype(np.float64).T / math.sqrt(D) + mask
        a = softmax(logits, axis=-1)
        exp_imp[h] += a.sum(0) / G
        other = m[0][None, :] != m[0][pos][:, None]
        assert abs(cross[0, g] - a[other].sum()) < 1e-12
    np.testing.assert_allclose(imp[0], exp_imp, rtol=1e-11, atol=1e-15)


def test_whole_prompt_as_window_is_the_full_prefill_flow():
    """With the window equal to the prompt every query row is a proxy row, and the masses of Eq. 7 are the literal
    sums over all (query, key) pairs, text-to-visual and visual-to-text: checked against scipy's causal softmax,
    against the uniform-attention closed form, and against the two one-modality cases."""
    rng = np.random.default_rng(29)
    L, D = 37, 16
    p = params(Hq=2, Hkv=1, D=D, L=L, W=L, B=1)
    q, k, v, m = rand_unit(rng, p, vis_frac=0.5)
    _, cross, total = O.score(p, q, k, m)
    mask = np.where(np.arange(L)[None, :] <= np.arange(L)[:, None], 0.0, -np.inf)
    other = m[0][None, :] != m[0][:, None]
    for g in range(2):
        a = softmax(q[0, g].astype(np.float64) @ k[0, 0].astype(np.float64).T / math.sqrt(D) + mask, axis=-1)
        v2t = a[(m[0] == 1)[:, None] & (m[0] == 0)[None, :]].sum()       # visual queries on text keys
        t2v = a[(m[0] == 0)[:, None] & (m[0] == 1)[None, :]].sum()
        assert abs(cross[0, g] - (v2t + t2v)) < 1e-12 and abs(cross[0, g] - a[other].sum()) < 1e-12
        assert abs(total[0, g] - L) < 1e-12
    q[:] = 0                                                             # uniform rows: alpha[j, i] = 1 / (j + 1)
    _, cross, _ = O.score(p, q, k, m)
    exp = sum(Fraction(sum(1 for i in range(j + 1) if m[0, i] != m[0, j]), j + 1) for j in range(L))
    np.testing.assert_allclose(cross[0], float(exp), rtol=1e-13)
    for vis in (0, 1):
        _, cross, total = O.score(p, rng.standard_normal(q.shape).astype(np.float32), k, np.full_like(m, vis))
        rho, strat = O.layer_flow(p, cross, total)
        assert np.all(cross == 0) and rho[0] == 0 and strat[0] == O.INTRA


def test_score_invariants():
    rng = np.random.default_rng(2)
    for (Hq, Hkv, D, L, W) in [(4, 2, 8, 37, 5), (3, 3, 16, 64, 64), (8, 1, 4, 19, 1)]:
        p = params(U=2, Hq=Hq, Hkv=Hkv, D=D, L=L, W=W, B=3)
        q, k, v, m = rand_unit(rng, p)
        imp, cross, total = O.score(p, q, k, m)
        assert np.all(imp >= 0)
        np.testing.assert_allclose(imp.sum(-1), W, rtol=1e-12)      # every softmax row sums to one
        np.testing.assert_allclose(total, W, rtol=1e-12)
        rho, strat = O.layer_flow(p, cross, total)
        assert np.all((rho >= 0) & (rho <= 1))
        # a single-modality prompt has no cross-modal flow
        for val in (0, 1):
            m1 = np.full_like(m, val)
            _, c1, t1 = O.score(p, q, k, m1)
            r1, s1 = O.layer_flow(p, c1, t1)
            assert np.all(c1 == 0) and np.all(r1 == 0) and np.all(s1 == O.INTRA)


def test_causal_mask_future_keys_do_not_matter():
    """Changing a key after a window row's position leaves that row's attention unchanged;
    with W = 1 only the last key is after nothing, so perturb inside the window."""
    rng = np.random.default_rng(3)
    p = params(Hq=1, Hkv=1, D=4, L=12, W=4, B=2)
    q, k, v, m = rand_unit(rng, p)
    imp0, _, _ = O.score(p, q, k, m)
    # the last key is visible to the last window row only
    k2 = k.copy(); k2[0, 0, -1] += 3.0
    q2 = q.copy(); q2[0, 0, -1] = 0.0   # last row uniform -> its attention ignores key values
    a, _, _ = O.score(p, q2, k, m)
    b, _, _ = O.score(p, q2, k2, m)
    np.testing.assert_allclose(a, b, rtol=1e-13)
    assert not np.allclose(imp0, O.score(p, q, k2, m)[0])


def test_flow_threshold_rule():
    p = params(U=3, Hq=2, theta=0.25)
    cross = np.array([[0.2, 0.3], [0.5, 0.5], [1.0, 0.2]])   # rho = .25, .5, .6 with total 1
    total = np.ones((3, 2))
    rho, strat = O.layer_flow(p, cross, total)
    np.testing.assert_allclose(rho, [0.25, 0.5, 0.6])
    assert strat.tolist() == [O.INTRA, O.CROSS, O.CROSS]     # equality is the conservative choice
    p.flow_mode = O.FLOW_FORCE_INTRA
    assert O.layer_flow(p, cross, total)[1].tolist() == [0, 0, 0]
    p.flow_mode = O.FLOW_FORCE_CROSS
    assert O.layer_flow(p, cross, total)[1].tolist() == [1, 1, 1]
    p.flow_mode = O.FLOW_MISALIGNED                          # the reverse of the rule, layer by layer
    assert O.layer_flow(p, cross, total)[1].tolist() == [O.CROSS, O.INTRA, O.INTRA]
    # head mean of ratios, not ratio of sums
    rho2, _ = O.layer_flow(params(U=1, Hq=2), np.array([[1.0, 0.0]]), np.array([[2.0, 8.0]]))
    assert abs(rho2[0] - 0.25) < 1e-15


# ---------------------------------------------------------------- select

def test_select_brute_force():
    rng = np.random.default_rng(7)
    for L, B in [(6, 1), (9, 4), (10, 10), (12, 5)]:
        p = params(Hq=2, Hkv=2, L=L, W=2, B=B)
        imp = rng.random((1, 2, L))
        ret, evi = O.select(p, imp)
        for h in range(2):
            best = max(itertools.combinations(range(L), B), key=lambda s: imp[0, h, list(s)].sum())
            assert ret[0, h].tolist() == sorted(best)
            assert evi[0, h].tolist() == sorted(set(range(L)) - set(best))
            if B < L:
                assert imp[0, h, ret[0, h]].min() >= imp[0, h, evi[0, h]].max()


def test_select_ties_and_keep_window():
    p = params(Hq=1, Hkv=1, L=8, W=3, B=3)
    imp = np.array([[[0.5, 0.9, 0.5, 0.5, 0.1, 0.5, 0.0, 0.2]]])
    ret, evi = O.select(p, imp)
    assert ret[0, 0].tolist() == [0, 1, 2]            # 0.9 first, then the lowest-index 0.5s
    assert evi[0, 0].tolist() == [3, 4, 5, 6, 7]
    p.keep_window = 1
    ret, _ = O.select(p, imp)
    assert ret[0, 0].tolist() == [5, 6, 7]            # the window fills the whole budget
    p.n_keep = 5
    ret, _ = O.select(p, imp)
    assert ret[0, 0].tolist() == [0, 1, 5, 6, 7]
    p.n_keep = 2
    with pytest.raises(ValueError):
        O.select(p, imp)


# ---------------------------------------------------------------- match

def _setup_match(rng, L=40, B=9, D=16, Hkv=2, vis_frac=0.5, **kw):
    p = params(Hq=Hkv, Hkv=Hkv, D=D, L=L, W=4, B=B, **kw)
    q, k, v, m = rand_unit(rng, p, vis_frac)
    imp = rng.random((1, Hkv, L))
    ret, evi = O.select(p, imp)
    return p, k, v, m, imp, ret, evi


def test_cosine_against_sklearn():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((6, 32)).astype(np.float32)
    ref = cosine_similarity(x.astype(np.float64))
    for i in range(6):
        for j in range(6):
            assert abs(O.cosine(x[i], x[j]) - ref[i, j]) < 1e-14
    assert O.cosine(np.zeros(32), x[0]) == 0.0


def test_match_ungated_is_nearest_centre():
    """tau = inf and a cross-modal layer: Eq. 10 is nearest-centre assignment; on unit-norm
    rows the nearest centre in Euclidean distance (scipy vq) is the one of largest cosine."""
    rng = np.random.default_rng(4)
    p, k, v, m, imp, ret, evi = _setup_match(rng, L=60, B=11, D=24)
    mt, sim, ru = O.match(p, k, imp, m, ret, evi, np.array([O.CROSS], dtype=np.int32))
    for h in range(p.n_kv_heads):
        kn = k[0, h].astype(np.float64)
        kn /= np.linalg.norm(kn, axis=1, keepdims=True)
        code, _ = vq(kn[evi[0, h]], kn[ret[0, h]])
        assert mt[0, h].tolist() == code.tolist()
        u = cosine_similarity(k[0, h][evi[0, h]].astype(np.float64), k[0, h][ret[0, h]].astype(np.float64))
        np.testing.assert_allclose(sim[0, h], u.max(1), rtol=1e-13)
        np.testing.assert_allclose(ru[0, h], np.sort(u, axis=1)[:, -2], rtol=1e-13)
        assert np.all((sim >= -1 - 1e-12) & (sim <= 1 + 1e-12))


@pytest.mark.parametrize("strategy", [O.INTRA, O.CROSS])
def test_match_gates_brute_force(strategy):
    """Enumerate every pivot for every non-pivot with numpy's own cosine and apply both gates."""
    rng = np.random.default_rng(9 + strategy)
    p, k, v, m, imp, ret, evi = _setup_match(rng, L=30, B=8, D=8, tau=0.8, tau_mode=O.TAU_ABS)
    mt, sim, _ = O.match(p, k, imp, m, ret, evi, np.array([strategy], dtype=np.int32))
    some_gated = some_empty = False
    for h in range(p.n_kv_heads):
        K = k[0, h].astype(np.float64)
        for j, e in enumerate(evi[0, h]):
            best, ub = -1, None
            for s, r in enumerate(ret[0, h]):
                if imp[0, h, r] > 0.8:
                    some_gated = True
                    continue
                if strategy == O.INTRA and m[0, r] != m[0, e]:
                    continue
                u = float(K[e] @ K[r] / (np.linalg.norm(K[e]) * np.linalg.norm(K[r])))
                if ub is None or u > ub:
                    best, ub = s, u
            assert mt[0, h, j] == best
            if best < 0:
                some_empty = True
                assert sim[0, h, j] == 0.0
            else:
                assert abs(sim[0, h, j] - ub) < 1e-13
    assert some_gated


def test_match_no_admissible_pivot_and_relative_tau():
    rng = np.random.default_rng(21)
    p, k, v, m, imp, ret, evi = _setup_match(rng, L=20, B=4, D=8, tau=-1.0)
    mt, sim, _ = O.match(p, k, imp, m, ret, evi, np.array([O.CROSS], dtype=np.int32))
    assert np.all(mt == -1) and np.all(sim == 0)
    # relative tau is measured in units of W / L
    p.tau_mode, p.tau = O.TAU_REL, 0.5 * p.seq_len / p.window   # tau_eff = 0.5
    a = O.match(p, k, imp, m, ret, evi, np.array([O.CROSS], dtype=np.int32))
    p.tau_mode, p.tau = O.TAU_ABS, 0.5
    b = O.match(p, k, imp, m, ret, evi, np.array([O.CROSS], dtype=np.int32))
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    # all pivots of the other modality + intra-modal layer -> nothing to merge into
    m2 = np.zeros_like(m); m2[0, ret[0, 0]] = 1
    p.tau = np.inf
    mt2, _, _ = O.match(p, k, imp, m2, ret, evi, np.array([O.INTRA], dtype=np.int32))
    assert np.all(mt2[0, 0] == -1)


def test_match_duplicates_and_scale_invariance():
    rng = np.random.default_rng(13)
    p, k, v, m, imp, ret, evi = _setup_match(rng, L=24, B=6, D=8)
    h = 0
    e, r0, r1 = evi[0, h, 3], ret[0, h, 2], ret[0, h, 4]
    k[0, h, r1] = k[0, h, r0]          # two identical pivots
    k[0, h, e] = 2.5 * k[0, h, r0]     # a non-pivot parallel to both
    cross = np.array([O.CROSS], dtype=np.int32)
    mt, sim, ru = O.match(p, k, imp, m, ret, evi, cross)
    assert mt[0, h, 3] == 2 and abs(sim[0, h, 3] - 1.0) < 1e-12 and abs(ru[0, h, 3] - 1.0) < 1e-12
    scale = rng.uniform(0.1, 9.0, size=(1, p.n_kv_heads, p.seq_len, 1)).astype(np.float32)
    k2 = (k.astype(np.float64) * scale).astype(np.float32)
    # exact powers of two keep the float32 products exact, so the result is identical
    k3 = k * np.float32(4.0)
    mt3, sim3, _ = O.match(p, k3, imp, m, ret, evi, cross)
    assert np.array_equal(mt3, mt)
    np.testing.assert_allclose(sim3, sim, rtol=1e-13)
    mt2, sim2, _ = O.match(p, k2, imp, m, ret, evi, cross)
    np.testing.assert_allclose(sim2, sim, atol=1e-6)


# ---------------------------------------------------------------- merge

def _dense_merge_matrix(p, ret, evi, mt, sim, h):
    L, B = p.seq_len, p.n_keep
    M = np.zeros((B, L))
    for s, r in enumerate(ret[0, h]):
        M[s, r] = 1.0
    for j, e in enumerate(evi[0, h]):
        if mt[0, h, j] >= 0:
            M[mt[0, h, j], e] = 1.0 if p.merge_mode == O.MERGE_MEAN else math.exp(sim[0, h, j] - 1.0)
    return M / M.sum(1, keepdims=True)


@pytest.mark.parametrize("mode", [O.MERGE_EXPSIM, O.MERGE_MEAN])
def test_merge_is_row_stochastic_matrix_product(mode):
    rng = np.random.default_rng(17)
    p, k, v, m, imp, ret, evi = _setup_match(rng, L=33, B=7, D=8, tau=0.9, merge_mode=mode)
    mt, sim, _ = O.match(p, k, imp, m, ret, evi, np.array([O.INTRA], dtype=np.int32))
    ko, vo, z = O.merge(p, k, v, ret, evi, mt, sim)
    for h in range(p.n_kv_heads):
        M = _dense_merge_matrix(p, ret, evi, mt, sim, h)
        assert np.all(M >= 0) and np.allclose(M.sum(1), 1.0)
        assert np.all((M > 0).sum(0) <= 1)                       # a token feeds at most one slot
        np.testing.assert_allclose(ko[0, h], M @ k[0, h].astype(np.float64), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(vo[0, h], M @ v[0, h].astype(np.float64), rtol=1e-12, atol=1e-14)
        # convex hull per channel, and protected pivots pass through untouched
        for s, r in enumerate(ret[0, h]):
            src = [r] + [e for j, e in enumerate(evi[0, h]) if mt[0, h, j] == s]
            assert np.all(ko[0, h, s] <= k[0, h, src].max(0) + 1e-12)
            assert np.all(ko[0, h, s] >= k[0, h, src].min(0) - 1e-12)
            if len(src) == 1:
                assert np.array_equal(ko[0, h, s], k[0, h, r].astype(np.float64))
                assert np.array_equal(vo[0, h, s], v[0, h, r].astype(np.float64))
            if imp[0, h, r] > 0.9:
                assert len(src) == 1


def test_merge_mean_is_cluster_average():
    """Uniform weights: each slot is the plain mean of its pivot and its members."""
    rng = np.random.default_rng(19)
    p, k, v, m, imp, ret, evi = _setup_match(rng, L=50, B=5, D=6, merge_mode=O.MERGE_MEAN)
    mt, sim, _ = O.match(p, k, imp, m, ret, evi, np.array([O.CROSS], dtype=np.int32))
    ko, vo, z = O.merge(p, k, v, ret, evi, mt, sim)
    for h in range(p.n_kv_heads):
        for s, r in enumerate(ret[0, h]):
            members = [r] + evi[0, h][mt[0, h] == s].tolist()
            np.testing.assert_allclose(vo[0, h, s], v[0, h, members].astype(np.float64).mean(0), rtol=1e-12, atol=1e-14)
            assert z[0, h, s] == len(members)


def test_full_budget_is_identity_and_low_tau_is_pure_eviction():
    rng = np.random.default_rng(23)
    p = params(Hq=2, Hkv=2, D=8, L=21, W=3, B=21)
    q, k, v, m = rand_unit(rng, p)
    out = O.compress_layer(p, q, k, v, m)
    assert np.array_equal(out["k_out"], k.astype(np.float64)) and np.array_equal(out["v_out"], v.astype(np.float64))
    assert out["evicted"].shape[-1] == 0
    p = params(Hq=2, Hkv=2, D=8, L=21, W=3, B=6, tau=0.0)      # every pivot is "highly sensitive"
    out = O.compress_layer(p, q, k, v, m)
    assert np.all(out["match"] == -1)
    for h in range(2):
        assert np.array_equal(out["k_out"][0, h], k[0, h][out["retained"][0, h]].astype(np.float64))
        assert np.array_equal(out["v_out"][0, h], v[0, h][out["retained"][0, h]].astype(np.float64))
    assert out["k_out"].shape == (1, 2, 6, 8)


def test_compress_layer_invariants_and_forcing():
    rng = np.random.default_rng(29)
    p = params(U=2, Hq=4, Hkv=2, D=8, L=48, W=6, B=10, tau=2.0, tau_mode=O.TAU_REL, theta=0.4)
    q, k, v, m = rand_unit(rng, p)
    out = O.compress_layer(p, q, k, v, m)
    L, B = p.seq_len, p.n_keep
    tau_eff = 2.0 * p.window / L
    for u in range(2):
        for h in range(2):
            r, e = out["retained"][u, h], out["evicted"][u, h]
            assert len(r) == B and len(e) == L - B
            assert sorted(set(r) | set(e)) == list(range(L)) and not (set(r) & set(e))
            assert np.all(np.diff(r) > 0) and np.all(np.diff(e) > 0)
            mt = out["match"][u, h]
            assert np.all((mt >= -1) & (mt < B))
            hit = mt >= 0
            assert np.all(out["importance"][u, h][r[mt[hit]]] <= tau_eff)
            if out["strategy"][u] == O.INTRA:
                assert np.all(m[u][r[mt[hit]]] == m[u][e[hit]])
    # forcing the other strategy changes only what follows it
    forced = O.compress_layer(p, q, k, v, m, forced={"strategy": 1 - out["strategy"]})
    assert np.array_equal(forced["retained"], out["retained"])
    assert np.array_equal(forced["rho"], out["rho"])
    assert not np.array_equal(forced["match"], out["match"])
