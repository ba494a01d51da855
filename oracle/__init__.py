"""CPU oracle of the WISV verifier: test infrastructure, never part of the product path."""
from .wisv_oracle import (  # noqa: F401
    ACT_GELU, ACT_RELU, build, head, hidden_as_f32, lm_head, scan, threads, verify,
)
