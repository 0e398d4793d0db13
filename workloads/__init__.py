"""Seeded synthetic inputs and shape descriptions.

This package serves both the CPU oracle and the CUDA library with the same
bytes.  It contains no arithmetic of the zeroth-order method itself: only
shape records, a storage-format helper (bf16 rounding) and calls to numpy's
own random generators.
"""
from .spec import ModelSpec, CONFIGS, config  # noqa: F401
from .synth import (  # noqa: F401
    bf16_round, to_bf16_bits, from_bf16_bits, make_linear_problem,
    make_decoder_problem, make_ragged_batch, make_decoder_globals, make_decoder_layer, next_token_labels, label_word_labels,
)
from .quant import quantize_int8, quantize_nf4, quantize_layer  # noqa: F401
