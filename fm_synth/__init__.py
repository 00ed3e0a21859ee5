"""Seeded synthetic inputs for the hourglass speculative-decode path.

This module only *draws data*: model hyper-parameters, random-init weights,
conditioning vectors, prompts and acceptance schedules.  It contains none of
the method's arithmetic (no attention, no norms, no hourglass, no decoding) so
that the CPU oracle and the CUDA library can both be fed from it without
sharing any code of the method itself.
"""
from .configs import CONFIGS, ModelConfig, get_config, toy_config
from .weights import make_weights, round_to_bf16, stack_names
from .inputs import (make_condition, make_prompt, icosphere_faces,
                     accept_schedule, stop_lengths, fill_prompt)

__all__ = ["CONFIGS", "ModelConfig", "get_config", "toy_config", "make_weights",
           "round_to_bf16", "stack_names", "make_condition", "make_prompt",
           "icosphere_faces", "accept_schedule", "stop_lengths", "fill_prompt"]
