"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

Holds only input recipes: model shapes, weight draws, prompts and the controlled
draft table. None of the decoder's arithmetic lives here, and this module imports
neither the oracle nor the CUDA binding.
"""
from .configs import ModelConfig, CONFIGS, get_config  # noqa: F401
from .weights import tensor_specs, draw_tensor, draw_weights  # noqa: F401
from .prompts import draw_prompt, draw_prompt_batch, controlled_draft  # noqa: F401
from .device import stream_weights_to_device  # noqa: F401
