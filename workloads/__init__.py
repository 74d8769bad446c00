"""Seeded synthetic inputs for the superposition-prompting hot path.

This package holds only shapes, packing and random draws.  It contains none of
the method's arithmetic (no positions, no RoPE, no attention, no scores): the
CPU oracle and the CUDA library each implement those on their own and both are
fed from here.
"""
from .configs import CONFIGS, Config, get_config  # noqa: F401
from .layout import Layout, build_layout, draw_lengths, next_round_layout  # noqa: F401
from .tensors import (  # noqa: F401
    bf16_round,
    draw_decode_inputs,
    draw_logits,
    draw_prior_weight,
    draw_qkv,
    draw_targets,
)
