"""Seeded synthetic workloads (shapes and value distributions only).

This package holds none of the method's arithmetic: it only draws the random
key / value / query tensors that both the CUDA path and the CPU oracle are fed.
"""
from .synth import (CONFIGS, D_MODEL, WorkloadConfig, make_hidden_states, make_layer_kv,  # noqa: F401
                    make_saliency, make_step_inputs)
