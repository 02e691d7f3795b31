"""Seeded synthetic inputs for the FlowMM compression path.

The paper evaluates on MileBench prompts run through pretrained MLLMs; neither
is available here, so these generators stand in for a prefill result: per
(layer, sequence) unit they draw the layer's keys K, values V, the
observation-window queries Q and the text/visual modality map, with the
structure the paper describes (a distribution gap between modalities, shallow
layers attending mostly within a modality and deep layers across modalities).

Recipe, per unit (layer l, sequence s), KV head h, token i, channel c, with
z ~ N(0, 1) independent:
  * K[h, i, c] = z                      for a text token,
                 T_l * (0.5 + 1.5 z)    for a visual token (T_l: optional
                                        per-layer visual temperature);
    V likewise with T_l = 1.
  * optional outlier channels: a few channels per head multiplied by 8 in K;
  * optional heavy tails: a few channels per head drawn from Student-t(3);
  * optional video structure: consecutive visual runs are frames, and the
    underlying z of a frame is AR(1)-correlated with the previous frame at the
    same in-frame position;
  * Q[g, a, c] = z + s_a * beta_l / sqrt(D) on the Gaussian channels (no offset
    on heavy-tailed ones), s_a = +1 for a text window token and -1 for a visual
    one: the shared offset moves every visual logit by about 0.5 * s_a * beta_l,
    so a negative beta_l keeps a window token's attention inside its own
    modality and beta_l near zero lets it spread; beta_l ramps linearly from
    `beta_lo` at the first layer to `beta_hi` at the last.
For bf16 workloads every array is rounded to bf16 (round to nearest even) once
here, and returned as float32 holding exactly those values, so that every
consumer sees identical numbers.

Nothing in this module is part of the compression method: it only makes
inputs.  Two backends share the recipe: `make_unit` (numpy, Philox counter
RNG keyed by (seed, layer, sequence); the canonical one used wherever two
implementations are compared) and `make_stack_device` (torch RNG on a device,
for filling a whole stack quickly when timing).
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Sequence

import numpy as np

from .configs import TEXT, VISUAL, Workload


def modality_map(wl: Workload) -> np.ndarray:
    """uint8[L]: 0 = text, 1 = visual, in prompt order."""
    parts = [np.full(n, m, dtype=np.uint8) for m, n in wl.segments]
    return np.concatenate(parts)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def layer_beta(wl: Workload, layer: int) -> float:
    if wl.n_layers == 1:
        return wl.beta_lo
    return wl.beta_lo + (wl.beta_hi - wl.beta_lo) * layer / (wl.n_layers - 1)


def layer_visual_temp(wl: Workload, layer: int) -> float:
    if wl.n_layers == 1:
        return wl.visual_temp_lo
    return wl.visual_temp_lo + (wl.visual_temp_hi - wl.visual_temp_lo) * layer / (wl.n_layers - 1)


def _rng(wl: Workload, layer: int, seq: int) -> np.random.Generator:
    key = np.array([wl.seed, layer * 65536 + seq], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _frame_slices(wl: Workload):
    """Start/stop of every visual run, in prompt order."""
    out, pos = [], 0
    for m, n in wl.segments:
        if m == VISUAL:
            out.append((pos, pos + n))
        pos += n
    return out


def _base_noise(wl: Workload, rng: np.random.Generator, heads: int) -> np.ndarray:
    L, D = wl.seq_len, wl.head_dim
    z = rng.standard_normal((heads, L, D), dtype=np.float32)
    if wl.ar1_frames > 0:
        rho = wl.ar1_rho
        innov = math.sqrt(1.0 - rho * rho)
        frames = _frame_slices(wl)
        for f in range(1, len(frames)):
            a0, a1 = frames[f - 1]
            b0, b1 = frames[f]
            n = min(a1 - a0, b1 - b0)
            z[:, b0:b0 + n, :] = rho * z[:, a0:a0 + n, :] + innov * z[:, b0:b0 + n, :]
    return z


def make_unit(wl: Workload, layer: int, seq: int = 0) -> Dict[str, np.ndarray]:
    """One (layer, sequence) unit: q [Hq, W, D], k, v [Hkv, L, D] float32, modality uint8[L]."""
    L, D, W = wl.seq_len, wl.head_dim, wl.window
    Hq, Hkv = wl.n_q_heads, wl.n_kv_heads
    rng = _rng(wl, layer, seq)
    m = modality_map(wl)
    vis = (m == VISUAL)

    zk = _base_noise(wl, rng, Hkv)
    zv = _base_noise(wl, rng, Hkv)
    gauss = np.ones((Hkv, D), dtype=np.float32)    # 1 where a channel is Gaussian, 0 where heavy-tailed
    if wl.student_t_channels > 0:
        for h in range(Hkv):
            ch = rng.choice(D, size=wl.student_t_channels, replace=False)
            zk[h][:, ch] = rng.standard_t(3.0, size=(L, len(ch))).astype(np.float32)
            zv[h][:, ch] = rng.standard_t(3.0, size=(L, len(ch))).astype(np.float32)
            gauss[h, ch] = 0.0
    temp = np.float32(layer_visual_temp(wl, layer))
    k = zk.copy()
    v = zv.copy()
    k[:, vis, :] = temp * (np.float32(0.5) + np.float32(1.5) * zk[:, vis, :])
    v[:, vis, :] = np.float32(0.5) + np.float32(1.5) * zv[:, vis, :]
    if wl.outlier_channels > 0:
        for h in range(Hkv):
            ch = rng.choice(D, size=wl.outlier_channels, replace=False)
            k[h][:, ch] *= np.float32(8.0)
    beta = np.float32(layer_beta(wl, layer) / math.sqrt(D))
    sign = np.where(m[L - W:] == VISUAL, np.float32(-1.0), np.float32(1.0)).astype(np.float32)   # [W]
    offset = beta * sign[None, :, None] * np.repeat(gauss, wl.group, axis=0)[:, None, :]        # [Hq, W, D]
    q = rng.standard_normal((Hq, W, D), dtype=np.float32) + offset
    if wl.dtype == "bf16":
        q, k, v = round_to_bf16(q), round_to_bf16(k), round_to_bf16(v)
    return {"q": q, "k": k, "v": v, "modality": m}


def make_units(wl: Workload, units: Sequence[tuple]) -> Dict[str, np.ndarray]:
    """Stack several (layer, seq) units along a leading axis; modality becomes [U, L]."""
    parts = [make_unit(wl, layer, seq) for layer, seq in units]
    return {key: np.stack([p[key] for p in parts]) for key in ("q", "k", "v", "modality")}


def all_units(wl: Workload):
    return [(layer, seq) for layer in range(wl.n_layers) for seq in range(wl.n_seqs)]


def make_stack_device(wl: Workload, device, units: Optional[Sequence[tuple]] = None, seed_offset: int = 0):
    """Same recipe as `make_unit`, drawn with torch's RNG on `device`, for whole stacks.

    Returns torch tensors q [U, Hq, W, D], k, v [U, Hkv, L, D] in the workload's
    dtype and modality uint8 [U, L].  The random stream differs from the numpy
    backend; the distribution and structure are the same.
    """
    import torch

    units = list(units) if units is not None else all_units(wl)
    U, L, D, W = len(units), wl.seq_len, wl.head_dim, wl.window
    Hq, Hkv = wl.n_q_heads, wl.n_kv_heads
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    dev = torch.device(device)
    q = torch.empty((U, Hq, W, D), dtype=tdt, device=dev)
    k = torch.empty((U, Hkv, L, D), dtype=tdt, device=dev)
    v = torch.empty((U, Hkv, L, D), dtype=tdt, device=dev)
    m_np = modality_map(wl)
    m = torch.from_numpy(m_np).to(dev)
    vis = m.bool()
    frames = _frame_slices(wl)
    gen = torch.Generator(device=dev)
    sign = torch.where(vis[L - W:], -1.0, 1.0).to(torch.float32)

    def base(heads):
        z = torch.randn((heads, L, D), generator=gen, device=dev, dtype=torch.float32)
        if wl.ar1_frames > 0:
            rho = wl.ar1_rho
            innov = math.sqrt(1.0 - rho * rho)
            for f in range(1, len(frames)):
                a0, a1 = frames[f - 1]
                b0, b1 = frames[f]
                n = min(a1 - a0, b1 - b0)
                z[:, b0:b0 + n] = rho * z[:, a0:a0 + n] + innov * z[:, b0:b0 + n]
        return z

    def student_t3(shape):
        # t(3) = N(0,1) / sqrt(chi2(3) / 3)
        num = torch.randn(shape, generator=gen, device=dev)
        den = torch.randn(shape + (3,), generator=gen, device=dev).square().sum(-1).div(3.0).sqrt()
        return num / den

    for ui, (layer, seq) in enumerate(units):
        gen.manual_seed((wl.seed * 1000003 + layer * 65536 + seq + seed_offset * 7919) & 0x7FFFFFFF)
        zk, zv = base(Hkv), base(Hkv)
        gauss = torch.ones((Hkv, D), device=dev)
        if wl.student_t_channels > 0:
            for h in range(Hkv):
                ch = torch.randperm(D, generator=gen, device=dev)[: wl.student_t_channels]
                zk[h][:, ch] = student_t3((L, wl.student_t_channels))
                zv[h][:, ch] = student_t3((L, wl.student_t_channels))
                gauss[h, ch] = 0.0
        temp = layer_visual_temp(wl, layer)
        kk, vv = zk.clone(), zv.clone()
        kk[:, vis] = temp * (0.5 + 1.5 * zk[:, vis])
        vv[:, vis] = 0.5 + 1.5 * zv[:, vis]
        if wl.outlier_channels > 0:
            for h in range(Hkv):
                ch = torch.randperm(D, generator=gen, device=dev)[: wl.outlier_channels]
                kk[h][:, ch] *= 8.0
        beta = layer_beta(wl, layer) / math.sqrt(D)
        offset = beta * sign[None, :, None] * gauss.repeat_interleave(wl.group, dim=0)[:, None, :]
        qq = torch.randn((Hq, W, D), generator=gen, device=dev, dtype=torch.float32) + offset
        q[ui], k[ui], v[ui] = qq.to(tdt), kk.to(tdt), vv.to(tdt)
    modality = m.unsqueeze(0).expand(U, L).contiguous()
    return q, k, v, modality
