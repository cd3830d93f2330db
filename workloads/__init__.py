"""Seeded synthetic inputs for the batched verification pass.

This package only *draws* inputs (model tensors, token ids, context K/V, page
assignments). It contains none of the method's arithmetic: no norm, no
attention, no softmax, no gate. Both the CPU oracle's tests and the CUDA
path's tests/bench feed from here so that they see identical bits.
"""
from .configs import (ModelShape, VerifyConfig, CascadeConfig, CONFIGS, CASCADES, get_config, get_cascade,
                      scaled_config)
from .generate import (
    bf16_bits_from_f32,
    e4m3_codes_from_f32,
    e5m2_codes_from_f32,
    model_weights,
    plant_verdict_rows,
    make_batch,
    context_kv,
    page_assignment,
    Batch,
)

__all__ = [
    "ModelShape", "VerifyConfig", "CascadeConfig", "CONFIGS", "CASCADES", "get_config", "get_cascade",
    "scaled_config",
    "bf16_bits_from_f32", "e4m3_codes_from_f32", "e5m2_codes_from_f32", "model_weights", "plant_verdict_rows", "make_batch",
    "context_kv", "page_assignment", "Batch",
]
