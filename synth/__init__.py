"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests/bench.

This module only draws random numbers and lays them out in the shapes the DiT
workloads use.  It holds none of the method's arithmetic (no quantizer, no
normalisation, no sampler maths): both implementations receive the same bits
and do all of the computing themselves.

Random streams: numpy's counter-based Philox generator keyed by
(seed, crc32(tensor name)), so every named tensor is reproducible on its own
and independent of the order in which tensors are drawn.
"""
from .generators import (  # noqa: F401
    DiTConfig,
    DIT_S2_BLOCK,
    DIT_XL2,
    DIT_XL2_512,
    DIT_TINY,
    stream,
    normal,
    uniform_int,
    block_weights,
    model_weights,
    outlier_activations,
    pos_embed_table,
    CONFIG_SEEDS,
)
