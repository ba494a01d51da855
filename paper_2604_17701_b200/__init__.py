"""B200-native WISV edge-side verifier: thin Python binding over the C-ABI CUDA library.

Every step of the verification round runs inside ``libwisv.so`` (hand-written
sm_100a kernels).  This package only marshals arguments: torch supplies device
memory and the stream handle.  There is no CPU path; if the library is missing
or the device is not a B200, calls fail loudly.
"""
from .binding import (  # noqa: F401
    WisvError, Verifier, VerifyOutput, load_library, exported_symbols, lm_head_reduce_static,
    LinkParams, link_cost_round, choose_protocol, plan_host,
    ACT_RELU, ACT_GELU, MODE_FH, MODE_SH, ACCEPT_GREEDY, ACCEPT_STOCHASTIC, DT_F32, DT_BF16, DT_F16,
)
