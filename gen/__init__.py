"""Seeded synthetic inputs for the WISV edge-side verifier.

This module only draws random arrays and arranges them in the layouts the
verifier consumes.  It holds none of the verifier's arithmetic: anything that
depends on a model output (the reference argmax used to force draft-token
matches) is passed in by the caller.  Both the CPU oracle's tests and the CUDA
path's tests/bench consume these arrays, so the two sides see identical bytes.
"""
from .synth import (  # noqa: F401
    VerifyConfig,
    CONFIGS,
    config,
    make_weights,
    make_hidden,
    make_draft_tokens,
    make_stochastic_inputs,
    pack_selective,
    row_offsets,
    f32_to_bf16_bits,
    bf16_bits_to_f32,
)
