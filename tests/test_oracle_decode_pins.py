"""Pins for the oracle's decode-step attention (Eq. 4 over a cache): closed forms, invariants and a
library cross-check, so that a wrong index, sign or normaliser fails at least one of them."""
import numpy as np

from oracle import flowmm_oracle as O


def _rand(rng, U, Hq, Hkv, N, D):
    return (rng.standard_normal((U, Hq, D)).astype(np.float32), rng.standard_normal((U, Hkv, N, D)).astype(np.float32),
            rng.standard_normal((U, Hkv, N, D)).astype(np.float32))


def test_single_key_returns_its_value():
    rng = np.random.default_rng(0)
    q, k, v = _rand(rng, 2, 4, 2, 1, 16)
    out = O.decode_attention(q, k, v)
    for g in range(4):
        assert np.array_equal(out[:, g], v[:, g // 2, 0].astype(np.float64))


def test_equal_keys_give_the_mean_value_and_zero_query_too():
    rng = np.random.default_rng(1)
    q, k, v = _rand(rng, 1, 2, 1, 7, 8)
    k[:] = k[:, :, :1]                                   # all keys identical: uniform attention
    assert np.allclose(O.decode_attention(q, k, v), v.astype(np.float64).mean(2), atol=1e-12)
    q0, k1, v1 = _rand(rng, 1, 2, 1, 7, 8)
    q0[:] = 0                                            # zero query: uniform attention whatever the keys
    assert np.allclose(O.decode_attention(q0, k1, v1), np.broadcast_to(v1.astype(np.float64).mean(2), (1, 2, 8)), atol=1e-12)


def test_two_keys_closed_form_and_scale():
    # logits a and b: weights sigmoid(a - b) and its complement; head_dim 4 -> scale 1/2
    q = np.array([[[2.0, 0, 0, 0]]], dtype=np.float32)
    k = np.array([[[[1.0, 0, 0, 0], [-1.0, 0, 0, 0]]]], dtype=np.float32)
    v = np.array([[[[1.0, 0, 0, 0], [0, 1.0, 0, 0]]]], dtype=np.float32)
    out = O.decode_attention(q, k, v)
    w = 1.0 / (1.0 + np.exp(-2.0))                       # a - b = (2 - (-2)) / sqrt(4) = 2
    assert np.allclose(out[0, 0], [w, 1 - w, 0, 0], atol=1e-15)
    out1 = O.decode_attention(q, k, v, scale=1.0)        # explicit scale: a - b = 4
    w1 = 1.0 / (1.0 + np.exp(-4.0))
    assert np.allclose(out1[0, 0], [w1, 1 - w1, 0, 0], atol=1e-15)


def test_matches_numpy_softmax_with_gqa_mapping():
    rng = np.random.default_rng(2)
    U, Hq, Hkv, N, D = 2, 6, 2, 37, 16
    q, k, v = _rand(rng, U, Hq, Hkv, N, D)
    out = O.decode_attention(q, k, v)
    kk = np.repeat(k.astype(np.float64), Hq // Hkv, axis=1)      # query head g reads KV head g // G
    vv = np.repeat(v.astype(np.float64), Hq // Hkv, axis=1)
    s = np.einsum("ugd,ugnd->ugn", q.astype(np.float64), kk) / np.sqrt(D)
    a = np.exp(s - s.max(-1, keepdims=True))
    a /= a.sum(-1, keepdims=True)
    assert np.allclose(out, np.einsum("ugn,ugnd->ugd", a, vv), rtol=1e-12, atol=1e-12)


def test_invariances():
    rng = np.random.default_rng(3)
    q, k, v = _rand(rng, 1, 4, 4, 50, 8)
    ref = O.decode_attention(q, k, v)
    perm = rng.permutation(50)
    assert np.allclose(O.decode_attention(q, k[:, :, perm], v[:, :, perm]), ref, atol=1e-12)     # order of the cache
    lo, hi = v.min(2), v.max(2)
    assert np.all(ref >= lo - 1e-12) and np.all(ref <= hi + 1e-12)                               # convex combination
    # a key far below the others in logit gets no weight: dropping it changes nothing
    k2 = k.copy(); k2[:, :, 0] = -1e4 * q[:, :, :]
    assert np.allclose(O.decode_attention(q, k2, v), O.decode_attention(q, k2[:, :, 1:], v[:, :, 1:]), atol=1e-12)
