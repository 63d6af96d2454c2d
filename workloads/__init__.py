"""Seeded synthetic inputs for ChunkKV compression (no method arithmetic lives here)."""
from .synthetic import (  # noqa: F401
    CONFIGS,
    LayerInputs,
    Workload,
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    make_layer,
    iter_layers,
    ragged_lengths,
    scaled,
)
