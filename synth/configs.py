"""The five benchmark workloads: shapes, seeds and ST^3 hyper-parameters.

Shapes follow LLaVA-1.5-7B/13B and LLaVA-NeXT decoding (576 = 24x24 CLIP-L/14
patches at 336 px, 2880 = five such tiles, 35-token system prompt).  The
hyper-parameters S, R are the paper's chosen settings for 7B (S=7, R=12.25%)
and 13B (S=4, R=5%), P = 50%; tau is set to the number of decode steps so the
last step lands on beta = 0 (the tiny workload uses the paper's tau = 50).
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    batch: int
    num_layers: int
    num_heads: int
    head_dim: int
    dtype: str                    # "f32" | "bf16"
    sys_len: int
    num_visual: int
    text_len_min: int
    text_len_max: int             # per-sequence text length is uniform in [min, max]
    decode_steps: int
    first_prune_layer: int
    stride: int
    first_ratio_bp: int
    step_ratio_bp: int
    tau: float
    planted: str                  # "uniform" | "drift" | "patch"
    num_planted: int
    grid_side: int = 24           # visual tokens form tiles of grid_side x grid_side

    @property
    def max_text_len(self) -> int:
        return self.text_len_max

    @property
    def t0_max(self) -> int:
        return self.sys_len + self.num_visual + self.text_len_max

    def scaled(self, **kw) -> "Workload":
        """A copy with some fields replaced (smaller step counts for tests)."""
        return replace(self, **kw)


WORKLOADS = {
    "tiny": Workload(
        name="tiny", seed=0, batch=1, num_layers=1, num_heads=8, head_dim=64, dtype="f32",
        sys_len=32, num_visual=576, text_len_min=32, text_len_max=32, decode_steps=16,
        first_prune_layer=0, stride=1, first_ratio_bp=5000, step_ratio_bp=0, tau=50.0,
        planted="uniform", num_planted=32),
    "llava15_7b": Workload(
        name="llava15_7b", seed=1, batch=1, num_layers=32, num_heads=32, head_dim=128, dtype="bf16",
        sys_len=35, num_visual=576, text_len_min=64, text_len_max=64, decode_steps=256,
        first_prune_layer=3, stride=7, first_ratio_bp=5000, step_ratio_bp=1225, tau=256.0,
        planted="drift", num_planted=28),
    "llava15_7b_b32": Workload(
        name="llava15_7b_b32", seed=2, batch=32, num_layers=32, num_heads=32, head_dim=128, dtype="bf16",
        sys_len=35, num_visual=576, text_len_min=16, text_len_max=128, decode_steps=512,
        first_prune_layer=3, stride=7, first_ratio_bp=5000, step_ratio_bp=1225, tau=512.0,
        planted="drift", num_planted=28),
    "llava15_13b_b16": Workload(
        name="llava15_13b_b16", seed=3, batch=16, num_layers=40, num_heads=40, head_dim=128, dtype="bf16",
        sys_len=35, num_visual=576, text_len_min=64, text_len_max=64, decode_steps=512,
        first_prune_layer=3, stride=4, first_ratio_bp=5000, step_ratio_bp=500, tau=512.0,
        planted="drift", num_planted=28),
    "llava_next_b8": Workload(
        name="llava_next_b8", seed=4, batch=8, num_layers=32, num_heads=32, head_dim=128, dtype="bf16",
        sys_len=35, num_visual=2880, text_len_min=128, text_len_max=128, decode_steps=1024,
        first_prune_layer=3, stride=7, first_ratio_bp=5000, step_ratio_bp=1225, tau=1024.0,
        planted="patch", num_planted=86),
}

ORDER = ["tiny", "llava15_7b", "llava15_7b_b32", "llava15_13b_b16", "llava_next_b8"]


def get_workload(name_or_index) -> Workload:
    if isinstance(name_or_index, int):
        return WORKLOADS[ORDER[name_or_index]]
    return WORKLOADS[name_or_index]
