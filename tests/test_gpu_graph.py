"""The whole-stack call and the decode call are stream-ordered and allocation-free, so they can be
captured once in a CUDA graph and replayed: the replay must write the same bits as the plain call."""
import pytest
import torch

from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import configs, inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_capture_and_replay_whole_stack(name):
    wl = configs.get(name)
    units = [(l, 0) for l in range(0, wl.n_layers, 4)]
    U, B = len(units), wl.n_keep(100)
    p = F.Params(U, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, B, dtype=F.BF16,
                 theta=wl.theta, tau=wl.tau_rel, tau_mode=F.TAU_REL)
    q, k, v, m = inputs.make_stack_device(wl, "cuda", units)
    ws = F.alloc_workspace(p, "cuda")
    k_out = torch.empty((U, wl.n_kv_heads, B, wl.head_dim), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    q_dec = q[:, :, -1, :].contiguous()
    o_dec = torch.empty(q_dec.shape, dtype=torch.float32, device="cuda")
    ws_dec = torch.empty(F.flowmm_decode_workspace_bytes(q_dec, k_out, v_out), dtype=torch.uint8, device="cuda")

    def call():
        F.flowmm_compress_layer(p, q, k, v, m, k_out, v_out, ws)
        F.flowmm_decode_attention(q_dec, k_out, v_out, o_dec, ws_dec)

    call()
    torch.cuda.synchronize()
    ref = (k_out.clone(), v_out.clone(), o_dec.clone())
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        call()                                   # warm-up on the capturing stream (function attributes, symbol look-ups)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            call()
    for _ in range(2):
        k_out.zero_(); v_out.zero_(); o_dec.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert F.flowmm_last_device_status(ws) == 0 and F.flowmm_last_device_status(ws_dec) == 0
        assert torch.equal(k_out, ref[0]) and torch.equal(v_out, ref[1]) and torch.equal(o_dec, ref[2])
