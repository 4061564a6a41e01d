"""Seeded synthetic inputs for the TiDAR decode step.

This module serves both the CPU oracle and the CUDA path.  It holds no arithmetic
of the method itself: only a counter-based random generator (splitmix64 of
(seed, tensor id, element index)), a Box-Muller transform, and the model /
workload shape tables.  Every value is a pure function of (seed, tensor id,
index), so a tensor can be produced in chunks, on the host or on a device, and
either side can regenerate exactly the bytes the other one saw.
"""
from .generators import (  # noqa: F401
    CONFIGS,
    ModelShape,
    acceptance_schedule,
    gen_model_weights,
    gen_normal_bf16,
    gen_token_ids,
    splitmix64,
    tensor_id,
    uniform01,
)
from .lazy import LazyLayers, LazyRows, lazy_model_weights, production_seconds  # noqa: F401
