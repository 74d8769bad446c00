"""The five workload shapes.

Shapes stand in for the retrieval workloads the paper measures on (20 documents
per example, average document length 142.6 / 121.2 BPE tokens, Appendix D):
no dataset item is reproduced, only segment counts and length ranges.
"""
from __future__ import annotations

from dataclasses import dataclass

SEED_BASE = 20240410


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    n_prompts: int        # B
    n_heads: int          # H
    n_kv_heads: int       # H_kv
    head_dim: int         # D
    pre_len: int          # P
    n_docs: int           # N  (paths per prompt)
    doc_len_min: int      # L_i ~ U{min..max}
    doc_len_max: int
    qry_len: int          # Q
    vocab: int            # V
    top_k: int            # k
    decode_steps: int
    dtype: str            # "f32" | "bf16"
    qkv_std: float        # standard deviation of Q/K/V entries
    logit_std: float      # standard deviation of logits
    positions: str        # "integer" | "equilibrium"
    rope_base: float = 10000.0

    @property
    def seed(self) -> int:
        return SEED_BASE + self.index

    @property
    def elt_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


CONFIGS = (
    Config(0, "cfg0_tiny_f32", 1, 4, 4, 64, 16, 4, 32, 32, 8, 512, 1, 4,
           "f32", 1.0, 2.0, "integer"),
    Config(1, "cfg1_mpt7b_single", 1, 32, 32, 128, 32, 20, 96, 160, 24, 50432, 2, 64,
           "bf16", 128 ** -0.5, 3.0, "equilibrium"),
    Config(2, "cfg2_batched_serving", 64, 32, 32, 128, 32, 20, 64, 256, 24, 50432, 2, 32,
           "bf16", 128 ** -0.5, 3.0, "equilibrium"),
    Config(3, "cfg3_llama2_7b", 8, 32, 32, 128, 48, 100, 64, 256, 32, 32000, 4, 128,
           "bf16", 128 ** -0.5, 3.0, "equilibrium"),
    Config(4, "cfg4_long_context", 2, 32, 32, 128, 64, 400, 128, 512, 32, 32000, 8, 256,
           "bf16", 128 ** -0.5, 3.0, "equilibrium"),
)


def get_config(which) -> Config:
    if isinstance(which, Config):
        return which
    if isinstance(which, int):
        return CONFIGS[which]
    for c in CONFIGS:
        if c.name == which or c.name.split("_")[0] == which:
            return c
    raise KeyError(which)
