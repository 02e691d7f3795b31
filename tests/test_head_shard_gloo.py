"""Sharding a layer by KV head over two gloo ranks on CPU: each rank runs the path on its own heads, one
all-reduce of n_units floats carries rho, and the pieces put together equal the unsharded result.  The step
entry points are stood in for by the oracle here (no GPU); the ordering and the collective are the code under test."""
import dataclasses
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import shard


class OracleSteps:
    """The step entry points with the binding's signatures, computed by the oracle on CPU tensors."""

    @staticmethod
    def _op(p):
        return O.OracleParams(p.n_units, p.n_q_heads, p.n_kv_heads, p.head_dim, p.seq_len, p.window, p.n_keep,
                              theta=p.theta, tau=p.tau, tau_mode=p.tau_mode, flow_mode=p.flow_mode)

    def flowmm_score(self, p, q, k, m, imp, cross, ws):
        i, c, _ = O.score(self._op(p), q.numpy(), k.numpy(), m.numpy())
        imp.copy_(torch.from_numpy(i)); cross.copy_(torch.from_numpy(c))

    def flowmm_layer_flow(self, p, cross, rho, strat):
        c = cross.numpy().astype(np.float64)
        r, s = O.layer_flow(self._op(p), c, np.full_like(c, float(p.window)))   # a head's total mass is its window
        rho.copy_(torch.from_numpy(r)); strat.copy_(torch.from_numpy(s))

    def flowmm_select(self, p, imp, ret, evi, ws):
        r, e = O.select(self._op(p), imp.numpy())
        ret.copy_(torch.from_numpy(r)); evi.copy_(torch.from_numpy(e))

    def flowmm_match(self, p, k, imp, m, ret, evi, strat, match, sim, ws):
        mt, s, _ = O.match(self._op(p), k.numpy(), imp.numpy(), m.numpy(), ret.numpy(), evi.numpy(), strat.numpy())
        match.copy_(torch.from_numpy(mt)); sim.copy_(torch.from_numpy(s))

    def flowmm_merge(self, p, k, v, ret, evi, match, sim, ko, vo, ws):
        a, b = O.merge(self._op(p), k.numpy(), v.numpy(), ret.numpy(), evi.numpy(), match.numpy(), sim.numpy())[:2]
        ko.copy_(torch.from_numpy(a)); vo.copy_(torch.from_numpy(b))


def _problem():
    rng = np.random.default_rng(41)
    U, Hq, Hkv, D, L, W, B = 3, 4, 2, 16, 60, 6, 9
    q = rng.standard_normal((U, Hq, W, D)).astype(np.float32)
    k = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
    v = rng.standard_normal((U, Hkv, L, D)).astype(np.float32)
    m = (rng.random((U, L)) < 0.5).astype(np.uint8)
    # theta between the flow of the first rank's heads and the flow of the whole layer (unit 0), so that a rank on
    # its own would pick the other strategy there: only the mean over both ranks' heads gives the right one
    q[:, 2:] *= 3.0
    cross = O.score(O.OracleParams(U, Hq, Hkv, D, L, W, B), q, k, m)[1]
    theta = 0.5 * (cross[0].mean() + cross[0, :2].mean()) / W
    return U, Hq, Hkv, D, L, W, B, q, k, v, m, float(theta)


def _alloc(U, Hq, Hkv, D, L, B):
    E = L - B
    f64, i32 = torch.float64, torch.int32
    return {"importance": torch.zeros((U, Hkv, L), dtype=f64), "cross_mass": torch.zeros((U, Hq), dtype=f64),
            "rho": torch.zeros(U, dtype=f64), "strategy": torch.zeros(U, dtype=i32),
            "rho_local": torch.zeros(U, dtype=f64), "strategy_local": torch.zeros(U, dtype=i32),
            "retained": torch.zeros((U, Hkv, B), dtype=i32), "evicted": torch.zeros((U, Hkv, E), dtype=i32),
            "match": torch.zeros((U, Hkv, E), dtype=i32), "match_sim": torch.zeros((U, Hkv, E), dtype=f64),
            "k_out": torch.zeros((U, Hkv, B, D), dtype=f64), "v_out": torch.zeros((U, Hkv, B, D), dtype=f64)}


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        U, Hq, Hkv, D, L, W, B, q, k, v, m, theta = _problem()
        h0, h1 = shard.head_range(Hkv, rank, world)
        G = Hq // Hkv
        p_local = F.Params(U, (h1 - h0) * G, h1 - h0, D, L, W, B, dtype=F.F32, theta=theta, tau=4.0, tau_mode=F.TAU_REL)
        out = _alloc(U, (h1 - h0) * G, h1 - h0, D, L, B)
        t = torch.from_numpy
        shard.compress_layer_head_sharded(p_local, t(q[:, h0 * G:h1 * G].copy()), t(k[:, h0:h1].copy()), t(v[:, h0:h1].copy()),
                                          t(m), out, None, steps=OracleSteps())
        out_q.put((rank, {key: val.numpy() for key, val in out.items()}))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_by_kv_head_equal_the_unsharded_layer():
    ctx = mp.get_context("spawn")
    out_q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out_q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(out_q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    U, Hq, Hkv, D, L, W, B, q, k, v, m, theta = _problem()
    op = O.OracleParams(U, Hq, Hkv, D, L, W, B, theta=theta, tau=4.0, tau_mode=O.TAU_REL)
    ref = O.compress_layer(op, q, k, v, m)
    # the layer's rho is the mean over both ranks' heads, and both ranks hold it
    for r in (0, 1):
        np.testing.assert_allclose(got[r]["rho"], ref["rho"], rtol=1e-12)
        assert np.array_equal(got[r]["strategy"], ref["strategy"])
    for key in ("retained", "evicted", "match"):
        assert np.array_equal(np.concatenate([got[0][key], got[1][key]], axis=1), ref[key]), key
    for key in ("k_out", "v_out", "importance"):
        np.testing.assert_allclose(np.concatenate([got[0][key], got[1][key]], axis=1), ref[key], rtol=1e-12, atol=1e-15)
    # a rank on its own would have decided differently for at least one unit: the collective matters
    alone = [O.layer_flow(dataclasses.replace(op, n_q_heads=Hq // 2, n_kv_heads=1),
                          ref_cross, np.full_like(ref_cross, float(W)))[1]
             for ref_cross in (O.score(op, q, k, m)[1][:, :Hq // 2], O.score(op, q, k, m)[1][:, Hq // 2:])]
    assert any(not np.array_equal(a, ref["strategy"]) for a in alone)


def test_head_range():
    assert shard.head_range(8, 0, 4) == (0, 2) and shard.head_range(8, 3, 4) == (6, 8)
    with pytest.raises(ValueError):
        shard.head_range(6, 0, 4)
    with pytest.raises(ValueError):
        shard.head_range(8, 4, 4)
