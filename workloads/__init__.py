"""Seeded synthetic inputs: rollout trees and q/k/v/g/dO tensors.

This package is the one piece shared by the CPU oracle and the CUDA path.  It
holds input generation only -- tree shapes and random tensors -- and none of
the method's arithmetic (no recurrence, no planning, no chunking).
"""
from .trees import Forest, make_forest, CONFIGS, config_forest  # noqa: F401
from .tensors import make_inputs, make_gk, make_logits, make_logp_grad, make_conv_inputs, make_attn_inputs  # noqa: F401
