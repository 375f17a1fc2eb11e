"""Seeded synthetic workloads for the Encode stage: architecture tables, random-init
weights and media inputs.  Shared by the CPU oracle's tests and by the CUDA path's tests
and benchmark.  Holds data generation only: none of the encoder's arithmetic lives here."""
from .configs import CONFIGS, get_config, weight_shapes, tokens_per_item, out_tokens_per_item  # noqa: F401
from .generate import (round_to_bf16, make_weights, make_items, draw_item_shapes,  # noqa: F401
                       sinusoid_table, to_bf16_bits)
