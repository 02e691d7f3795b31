"""Helpers shared by the GPU tests: run the CUDA path on numpy inputs, hand back numpy outputs."""
import numpy as np
import torch

from oracle import flowmm_oracle as O
from paper_2511_05534_b200 import binding as F


def gpu_params(p: O.OracleParams, dtype: int, path: int = F.PATH_AUTO) -> F.Params:
    return F.Params(p.n_units, p.n_q_heads, p.n_kv_heads, p.head_dim, p.seq_len, p.window, p.n_keep, dtype=dtype,
                    softmax_scale=p.softmax_scale, theta=p.theta, tau=p.tau, tau_mode=p.tau_mode,
                    flow_mode=p.flow_mode, merge_mode=p.merge_mode, keep_window=p.keep_window, path=path)


def to_dev(x: np.ndarray, dtype: int) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(F.torch_dtype(dtype))


def run_gpu(p: O.OracleParams, q, k, v, modality, dtype: int, path: int = F.PATH_AUTO):
    """flowmm_compress_layer through the C ABI; every output as a numpy array."""
    fp = gpu_params(p, dtype, path)
    qd, kd, vd = to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype)
    md = torch.from_numpy(np.ascontiguousarray(modality, dtype=np.uint8)).to("cuda")
    out = F.compress_layer_alloc(fp, qd, kd, vd, md)
    status = F.flowmm_last_device_status(out["ws"])
    assert status == 0, F.status_string(status)
    res = {}
    for key, t in out.items():
        if key == "ws":
            continue
        res[key] = t.float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.cpu().numpy()
    return res


def oracle_params(wl, n_units: int, permille: int, **kw) -> O.OracleParams:
    base = dict(theta=wl.theta, tau=wl.tau_rel, tau_mode=O.TAU_REL)
    base.update(kw)
    return O.OracleParams(n_units, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window,
                          wl.n_keep(permille), **base)
