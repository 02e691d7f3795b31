"""Workload shapes for the FlowMM compression hot path.

Each `Workload` names the shape of one synthetic MLLM prefill result: how many
(layer, sequence) units there are, the attention-head layout, the interleaving
of text and visual tokens in the prompt, the observation-window length (the
proxy set of Eq. 8: the last W prompt positions) and the retention budgets.

This module holds shapes and generator constants only; it has no arithmetic of
the method.  The one formula here, `n_keep`, turns a budget in permille into
the integer pivot count B of Section 3.3.1 with integer arithmetic
(ceil(L * permille / 1000), at least 1), so that no float rounding can change B.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

TEXT = 0
VISUAL = 1


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_seqs: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                      # "f32" or "bf16"
    segments: Tuple[Tuple[int, int], ...]   # (modality, run length) in prompt order
    window: int
    budgets_permille: Tuple[int, ...]
    seed: int
    # generator constants (see inputs.py)
    beta_lo: float = -14.0          # visual-attention bias of the shallowest layer
    beta_hi: float = -2.0           # ... of the deepest layer
    tau_rel: float = 4.0            # sensitivity threshold in units of W / L
    outlier_channels: int = 0       # channels per KV head scaled x8 in K
    student_t_channels: int = 0     # channels per KV head drawn from Student-t(3)
    visual_temp_lo: float = 1.0     # per-layer scale on visual keys, first layer
    visual_temp_hi: float = 1.0     # ... last layer
    ar1_frames: int = 0             # >0: visual runs are frames correlated AR(1)
    ar1_rho: float = 0.9
    theta: float = 0.25

    @property
    def seq_len(self) -> int:
        return sum(n for _, n in self.segments)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_units(self) -> int:
        return self.n_layers * self.n_seqs

    def n_keep(self, permille: int) -> int:
        L = self.seq_len
        return max(1, (L * permille + 999) // 1000)


def _video_segments(frames: int, vis: int, txt: int) -> Tuple[Tuple[int, int], ...]:
    segs: List[Tuple[int, int]] = []
    for _ in range(frames):
        segs.append((VISUAL, vis))
        segs.append((TEXT, txt))
    return tuple(segs)


WORKLOADS: Dict[str, Workload] = {
    # small fp32 case the oracle finishes in well under a second
    "cfg1": Workload(
        name="cfg1", n_layers=1, n_seqs=1, n_q_heads=4, n_kv_heads=4, head_dim=64, dtype="f32",
        segments=((TEXT, 8), (VISUAL, 144), (TEXT, 40)), window=16, budgets_permille=(250,), seed=0,
        beta_lo=-6.0, beta_hi=-6.0),
    # LLaVA-1.5-7B-shaped stack (MHA)
    "cfg2": Workload(
        name="cfg2", n_layers=32, n_seqs=1, n_q_heads=32, n_kv_heads=32, head_dim=128, dtype="bf16",
        segments=((TEXT, 16), (VISUAL, 576), (TEXT, 48)), window=32, budgets_permille=(50, 100, 200), seed=1,
        outlier_channels=4, beta_lo=-24.0, beta_hi=-2.0, tau_rel=10.0),
    # Qwen2-VL-7B-shaped stack (GQA group 7), one dynamic-resolution image
    "cfg3": Workload(
        name="cfg3", n_layers=28, n_seqs=1, n_q_heads=28, n_kv_heads=4, head_dim=128, dtype="bf16",
        segments=((TEXT, 32), (VISUAL, 2048), (TEXT, 96)), window=32, budgets_permille=(100,), seed=2,
        visual_temp_lo=0.5, visual_temp_hi=2.0, beta_lo=-18.0, beta_hi=-2.0, tau_rel=10.0),
    # multi-image / video-shaped stack: 8 frames interleaved with text
    "cfg4": Workload(
        name="cfg4", n_layers=28, n_seqs=1, n_q_heads=28, n_kv_heads=4, head_dim=128, dtype="bf16",
        segments=_video_segments(8, 1024, 32), window=64, budgets_permille=(50, 200), seed=3,
        ar1_frames=8, beta_lo=-20.0, beta_hi=0.0, tau_rel=8.0),
    # long-context stress, 4 independent sequences
    "cfg5": Workload(
        name="cfg5", n_layers=80, n_seqs=4, n_q_heads=64, n_kv_heads=8, head_dim=128, dtype="bf16",
        segments=((TEXT, 128), (VISUAL, 32768), (TEXT, 896)), window=64, budgets_permille=(50,), seed=4,
        student_t_channels=8, beta_lo=-40.0, beta_hi=-4.0, tau_rel=4.0),
}


def get(name: str) -> Workload:
    return WORKLOADS[name]
