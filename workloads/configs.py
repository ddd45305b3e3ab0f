"""The five workloads: shapes of Llama-2 decoder-block linear layers (the
shapes the paper's Table "linear_speed" lists, plus the grouped-query k/v
projections of the 70B model), quantiser geometry, token counts and the value
distributions of the synthetic stand-ins for trained weights and activations.

Token counts follow the paper's training set-up (Sec. 4.1): Block-AP uses
batch 2 x context 2048, E2E-QP uses context 4096.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Tuple


@dataclass(frozen=True)
class Linear:
    name: str
    out_features: int
    in_features: int
    count: int = 1          # how many linears of this shape one decoder block has


@dataclass(frozen=True)
class Config:
    name: str
    linears: Tuple[Linear, ...]
    bits: int
    group: int
    tokens: int
    modes: Tuple[str, ...]            # "block_ap", "e2e_qp"
    weight_dist: str                  # "normal" | "student_t4"
    weight_scale: float
    outlier_frac: float = 0.0         # fraction of input channels scaled by outlier_gain
    outlier_gain: float = 10.0
    x_std: float = 1.0
    dy_std: float = 1e-2

    def flops_per_mode(self) -> int:
        """2*T*in*out per contraction, three contractions (Y, dX, dW or ds) per linear."""
        return sum(3 * 2 * self.tokens * l.in_features * l.out_features * l.count for l in self.linears)


LINEARS = {
    "7b": (Linear("qkvo", 4096, 4096, 4), Linear("gate_up", 11008, 4096, 2), Linear("down", 4096, 11008, 1)),
    "13b": (Linear("qkvo", 5120, 5120, 4), Linear("gate_up", 13824, 5120, 2), Linear("down", 5120, 13824, 1)),
    "70b": (Linear("qo", 8192, 8192, 2), Linear("kv", 1024, 8192, 2),
            Linear("gate_up", 28672, 8192, 2), Linear("down", 8192, 28672, 1)),
}

CONFIGS = (
    Config("c1_single_w2g64", (Linear("single", 512, 512, 1),), 2, 64, 256, ("block_ap",), "normal", 0.02),
    Config("c2_7b_w4g128_block_ap", LINEARS["7b"], 4, 128, 4096, ("block_ap",), "student_t4", 0.02, 0.01),
    Config("c3_7b_w2g64_e2e_qp", LINEARS["7b"], 2, 64, 16384, ("e2e_qp",), "normal", 0.02),
    Config("c4_13b_w3g128_e2e_qp", LINEARS["13b"], 3, 128, 8192, ("e2e_qp",), "student_t4", 0.02, 0.01),
    Config("c5_70b_w2g64_both", LINEARS["70b"], 2, 64, 8192, ("block_ap", "e2e_qp"), "student_t4", 0.015),
)


def get_config(name: str) -> Config:
    for c in CONFIGS:
        if c.name == name or c.name.split("_")[0] == name:
            return c
    raise KeyError(name)
