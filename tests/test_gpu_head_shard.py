"""The head-sharded ordering of the steps on a GPU, in a world of one rank (no collective partner): the same bits
as the fused call.  Two ranks are covered on CPU (tests/test_head_shard_gloo.py)."""
import pytest
import torch

from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs, shard

pytestmark = pytest.mark.gpu


def _alloc(fp):
    U, Hq, Hkv, L, B, E, D = fp.n_units, fp.n_q_heads, fp.n_kv_heads, fp.seq_len, fp.n_keep, fp.n_evict, fp.head_dim
    dev, i32 = "cuda", torch.int32
    return {"importance": torch.empty((U, Hkv, L), device=dev), "cross_mass": torch.empty((U, Hq), device=dev),
            "rho": torch.empty(U, device=dev), "strategy": torch.empty(U, dtype=i32, device=dev),
            "rho_local": torch.empty(U, device=dev), "strategy_local": torch.empty(U, dtype=i32, device=dev),
            "retained": torch.empty((U, Hkv, B), dtype=i32, device=dev), "evicted": torch.empty((U, Hkv, E), dtype=i32, device=dev),
            "match": torch.empty((U, Hkv, E), dtype=i32, device=dev), "match_sim": torch.empty((U, Hkv, E), device=dev),
            "k_out": torch.empty((U, Hkv, B, D), dtype=torch.bfloat16, device=dev),
            "v_out": torch.empty((U, Hkv, B, D), dtype=torch.bfloat16, device=dev)}


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_one_rank_equals_the_fused_call(name):
    wl = configs.get(name)
    units = [(3, 0), (wl.n_layers - 2, 0)]
    q, k, v, m = inputs.make_stack_device(wl, "cuda", units)
    fp = F.Params(len(units), wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, wl.n_keep(100),
                  dtype=F.BF16, theta=wl.theta, tau=wl.tau_rel, tau_mode=F.TAU_REL)
    full = F.compress_layer_alloc(fp, q, k, v, m)
    out = shard.compress_layer_head_sharded(fp, q, k, v, m, _alloc(fp), F.alloc_workspace(fp))
    for key in ("importance", "rho", "strategy", "retained", "evicted", "match", "match_sim", "k_out", "v_out"):
        assert torch.equal(out[key], full[key]), key
