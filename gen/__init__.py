"""Seeded synthetic inputs (Pythia-shaped) shared by the CPU oracle tests and the CUDA tests.

This package only draws random tensors and packs them to bf16 bit patterns.  It contains none of the
early-exit arithmetic (no LayerNorm, projection, softmax, thresholding, compaction or acceptance).
"""
from .synth import (  # noqa: F401
    CONFIGS,
    bf16_bits_from_f32,
    f32_from_bf16_bits,
    make_head,
    make_hidden,
    make_planting,
    make_config,
    make_dssd_hidden,
    random_token_case,
    make_calibration_set,
    make_markov_model,
)
