"""The five workload shapes (model shape, prompt/decode lengths, BUZZ policy, key statistics)."""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    batch: int
    q_heads: int
    kv_heads: int
    head_dim: int
    dtype: str            # "f32" | "bf16"
    prompt_min: int       # prompt length (ragged when prompt_max > prompt_min)
    prompt_max: int
    decode_steps: int
    sink: int
    window: int
    segment: int
    hitters: int
    budget: int
    keys: str             # "outlier" | "lowrank" | "ar1" | "docs"
    outlier_p: float = 0.0
    outlier_scale: float = 1.0
    seed: int = 0x42555A5A

    @property
    def group(self) -> int:
        return self.q_heads // self.kv_heads

    @property
    def threshold(self) -> int:
        """T: capacity of the middle region (budget = T + sink + window)."""
        return self.budget - self.sink - self.window


CONFIGS = {
    # tiny single-layer decode, fp32
    "C1": Workload("C1", 1, 1, 1, 1, 64, "f32", 512, 512, 256, 4, 64, 16, 1, 160,
                   "outlier", 0.05, 4.0, 0x42555A5A + 1),
    # Llama-2-7B-shaped stack, budget = 40 % of (4096 + 512)
    "C2": Workload("C2", 32, 8, 32, 32, 128, "bf16", 4096, 4096, 512, 4, 512, 8, 1, 1843,
                   "lowrank", 0.02, 3.0, 0x42555A5A + 2),
    # long-context summarisation shape
    "C3": Workload("C3", 32, 4, 32, 32, 128, "bf16", 32768, 32768, 1024, 4, 1024, 16, 2, 4096,
                   "ar1", 0.0, 1.0, 0x42555A5A + 3),
    # GQA Llama-3-8B shape
    "C4": Workload("C4", 32, 16, 32, 8, 128, "bf16", 8192, 8192, 512, 4, 512, 8, 1, 2048,
                   "outlier", 0.03, 4.0, 0x42555A5A + 4),
    # ragged multi-document QA serving batch
    "C5": Workload("C5", 32, 32, 32, 32, 128, "bf16", 8192, 16384, 256, 4, 512, 16, 1, 2048,
                   "docs", 0.0, 1.0, 0x42555A5A + 5),
}


def get(name: str) -> Workload:
    return CONFIGS[name]


def scaled(w: Workload, **overrides) -> Workload:
    """A copy of a workload with some fields replaced (smaller cases for parity tests)."""
    return dataclasses.replace(w, **overrides)
