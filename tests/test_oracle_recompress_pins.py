"""Pins for the oracle's re-compression of a cache that grew during decoding (Eq. 3 followed by Section 3.3
again): what the reading fixes independently of the function itself."""
import numpy as np
import pytest

from oracle import flowmm_oracle as O


def _rand(seed, U, Hq, Hkv, D, L, W):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((U, Hq, W, D)).astype(np.float32)
    k = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
    v = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
    return rng, q, k, v


def test_same_modality_in_every_head_is_the_compression_path():
    """Before any compression every head of a layer holds the same tokens; the re-compression then is the
    compression path itself, head for head (this fixes the head mapping and that rho is the layer's)."""
    U, Hq, Hkv, D, L, W, B = 2, 6, 3, 16, 60, 5, 17
    rng, q, k, v = _rand(1, U, Hq, Hkv, D, L, W)
    m = (rng.random((U, L)) < 0.5).astype(np.uint8)
    p = O.OracleParams(U, Hq, Hkv, D, L, W, B, theta=0.45, tau=2.5, tau_mode=O.TAU_REL)
    a = O.compress_layer(p, q, k, v, m)
    b = O.recompress(p, q, k, v, np.repeat(m[:, None, :], Hkv, axis=1))
    assert set(a["strategy"]) == {0, 1}                       # both rules occur in this draw
    for key in ("importance", "rho", "strategy", "retained", "evicted", "match", "match_sim", "k_out", "v_out"):
        assert np.array_equal(a[key], b[key]), key
    assert np.array_equal(b["row_modality_out"], np.take_along_axis(np.repeat(m[:, None, :], Hkv, axis=1),
                                                                    a["retained"].astype(np.int64), -1))


def test_rho_is_the_mean_over_all_heads_with_each_heads_own_rows():
    """Two KV heads whose rows have different modalities: rho is the mean over all query heads of each head's own
    cross-modal share (written out with numpy here), and the one strategy it gives binds both heads."""
    U, Hq, Hkv, D, L, W, B = 1, 4, 2, 8, 40, 4, 10
    rng, q, k, v = _rand(2, U, Hq, Hkv, D, L, W)
    m = np.zeros((U, Hkv, L), np.uint8)
    m[0, 0, :30] = 1                                          # head 0: mostly visual rows, text window
    m[0, 1, :4] = 1                                           # head 1: almost all text
    shares = []
    for g in range(Hq):
        h = g // (Hq // Hkv)
        s = q[0, g].astype(np.float64) @ k[0, h].astype(np.float64).T / np.sqrt(D)       # [W, L]
        for a in range(W):
            s[a, L - W + a + 1:] = -np.inf
        alpha = np.exp(s - s.max(1, keepdims=True))
        alpha /= alpha.sum(1, keepdims=True)
        other = m[0, h][None, :] != m[0, h][L - W:][:, None]
        shares.append((alpha * other).sum() / alpha.sum())
    rho = float(np.mean(shares))
    per_head = [np.mean(shares[:2]), np.mean(shares[2:])]
    assert per_head[0] > 0.3 > per_head[1]                    # the heads alone would disagree at theta = 0.3
    for theta, want in ((rho * 0.99, O.CROSS), (rho * 1.01, O.INTRA)):
        p = O.OracleParams(U, Hq, Hkv, D, L, W, B, theta=theta)
        out = O.recompress(p, q, k, v, m)
        assert abs(out["rho"][0] - rho) < 1e-12 and out["strategy"][0] == want
        if want == O.INTRA:                                    # both heads merge inside a modality only
            for h in range(Hkv):
                hit = out["match"][0, h] >= 0
                piv = out["retained"][0, h][out["match"][0, h][hit]]
                assert np.array_equal(m[0, h][piv], m[0, h][out["evicted"][0, h][hit]])


def test_full_budget_is_the_plain_append_of_eq3():
    """Compress a prompt, append T decoded rows (Eq. 3), re-compress with room for everything: the cache comes
    back row for row, appended rows at the end, modalities carried along."""
    U, Hq, Hkv, D, L, W, B, T = 1, 4, 2, 8, 50, 4, 12, 6
    rng, q, k, v = _rand(3, U, Hq, Hkv, D, L, W)
    m = (rng.random((U, L)) < 0.6).astype(np.uint8)
    first = O.compress_layer(O.OracleParams(U, Hq, Hkv, D, L, W, B, tau=3.0, tau_mode=O.TAU_REL), q, k, v, m)
    k_new = rng.standard_normal((U, Hkv, T, D)).astype(np.float32)
    v_new = rng.standard_normal((U, Hkv, T, D)).astype(np.float32)
    k_cache = np.concatenate([first["k_out"].astype(np.float32), k_new], axis=2)
    v_cache = np.concatenate([first["v_out"].astype(np.float32), v_new], axis=2)
    rm = np.concatenate([np.take_along_axis(np.repeat(m[:, None, :], Hkv, axis=1), first["retained"].astype(np.int64), -1),
                         np.zeros((U, Hkv, T), np.uint8)], axis=2)          # decoded tokens are text
    q2 = rng.standard_normal((U, Hq, W, D)).astype(np.float32)
    out = O.recompress(O.OracleParams(U, Hq, Hkv, D, B + T, W, B + T), q2, k_cache, v_cache, rm)
    assert np.array_equal(out["k_out"], k_cache.astype(np.float64)) and np.array_equal(out["v_out"], v_cache.astype(np.float64))
    assert np.array_equal(out["row_modality_out"], rm)
    assert np.array_equal(out["retained"][0, 0], np.arange(B + T))


def test_second_round_keeps_the_budget_and_stays_inside_its_sources():
    """Two rounds: every row of the second result is a convex combination of rows of the grown cache (per-channel
    bounds), exactly B' rows per head, protected pivots pass unchanged, row modalities follow the pivots."""
    U, Hq, Hkv, D, L, W, B, T, B2 = 2, 4, 2, 8, 64, 4, 20, 8, 14
    rng, q, k, v = _rand(4, U, Hq, Hkv, D, L, W)
    m = (rng.random((U, L)) < 0.5).astype(np.uint8)
    first = O.compress_layer(O.OracleParams(U, Hq, Hkv, D, L, W, B, theta=0.4), q, k, v, m)
    k_cache = np.concatenate([first["k_out"], rng.standard_normal((U, Hkv, T, D))], axis=2).astype(np.float32)
    v_cache = np.concatenate([first["v_out"], rng.standard_normal((U, Hkv, T, D))], axis=2).astype(np.float32)
    rm = np.concatenate([np.take_along_axis(np.repeat(m[:, None, :], Hkv, axis=1), first["retained"].astype(np.int64), -1),
                         np.zeros((U, Hkv, T), np.uint8)], axis=2)
    q2 = rng.standard_normal((U, Hq, W, D)).astype(np.float32)
    p2 = O.OracleParams(U, Hq, Hkv, D, B + T, W, B2, theta=0.4, tau=1.5, tau_mode=O.TAU_REL)
    out = O.recompress(p2, q2, k_cache, v_cache, rm)
    assert out["k_out"].shape == (U, Hkv, B2, D) and out["retained"].shape == (U, Hkv, B2)
    tau_eff = p2.tau * W / (B + T)
    protected = 0
    for u in range(U):
        for h in range(Hkv):
            ret, evi, mt = out["retained"][u, h], out["evicted"][u, h], out["match"][u, h]
            assert np.array_equal(out["row_modality_out"][u, h], rm[u, h][ret])
            for s in range(B2):
                src = np.concatenate([[ret[s]], evi[mt == s]])
                for cache, res in ((k_cache, out["k_out"]), (v_cache, out["v_out"])):
                    rows = cache[u, h][src].astype(np.float64)
                    assert np.all(res[u, h, s] <= rows.max(0) + 1e-12) and np.all(res[u, h, s] >= rows.min(0) - 1e-12)
                if out["importance"][u, h, ret[s]] > tau_eff:
                    protected += 1
                    assert np.array_equal(out["k_out"][u, h, s], k_cache[u, h, ret[s]].astype(np.float64))
    assert protected > 0
