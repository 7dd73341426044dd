"""Seeded synthetic inputs (model shapes, bf16 weights, KV caches) for the decode-step tests and bench.

This package is shared by the CPU oracle's tests and the CUDA path's tests.  It contains no part of
the decoder's arithmetic: only the shape table and a counter-based normal generator.
"""
from .configs import CONFIGS, DecoderConfig, GLOBAL_SEED
from .generate import (build_generator, first_token, make_kv, make_weights, normal_bf16, synth_u64,
                       bf16_to_f32, TensorRole)

__all__ = ["CONFIGS", "DecoderConfig", "GLOBAL_SEED", "build_generator", "first_token", "make_kv",
           "make_weights", "normal_bf16", "synth_u64", "bf16_to_f32", "TensorRole"]
