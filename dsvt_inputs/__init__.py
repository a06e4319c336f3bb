"""Seeded synthetic inputs (coords, features, weights) for the DSVT hot path.

Data only: this package holds none of the method's arithmetic (no window ids,
no sorting, no set rule, no attention).  Both the CPU oracle's tests and the
CUDA library's tests draw their inputs from here so that they see identical
bytes; neither side's code lives here.
"""
from .configs import (  # noqa: F401
    CONFIG_IDS,
    bf16_bits,
    make_config,
    make_layer,
    make_pool_weights,
    random_case,
    round_bf16,
    unique_cells,
)
