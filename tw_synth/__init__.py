"""Seeded synthetic RNN-T models and encoder outputs.

This package only draws random numbers and shapes them into the tensors an
RNN-T decoder consumes (weights, embeddings, encoder frames, utterance
lengths).  It holds none of the search arithmetic: both the CPU oracle's
tests and the CUDA path's tests feed from it, and it imports neither.
"""
from .configs import CONFIGS, WorkloadConfig, get_config
from .generate import SyntheticModel, make_model, make_encoder_batch, round_to_bf16

__all__ = [
    "CONFIGS", "WorkloadConfig", "get_config",
    "SyntheticModel", "make_model", "make_encoder_batch", "round_to_bf16",
]
