"""Seeded synthetic inputs for the IODF integer flow: images, pruned model shapes, int8 weights and
requantisation parameters, and the entropy coder's prior tables.

This module only draws numbers and arranges them in plain numpy arrays. It holds none of the
method's arithmetic (no convolution, no requantisation, no coupling): the CPU oracle and the CUDA
library each marshal the arrays produced here into their own formats.
"""
from .rng import Stream
from .images import smooth_field_images
from .codec import logistic_codec
from .model import (make_model, make_residual_model, CONFIGS, config_model, config_images, model_macs, level_shapes,
                    latent_sizes, masked_dense_model, zero_padded_model)

__all__ = ["Stream", "smooth_field_images", "make_model", "make_residual_model", "CONFIGS", "config_model",
           "config_images", "model_macs", "level_shapes", "latent_sizes", "masked_dense_model",
           "zero_padded_model", "logistic_codec"]
