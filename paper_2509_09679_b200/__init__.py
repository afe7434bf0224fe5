"""B200-native butterfly rotation + low-bit quantization (ButterflyQuant hot path).

`Plan` wraps the C-ABI library `libbfq.so` (hand-written CUDA for sm_100a); `synth`
draws the seeded synthetic workloads.  Importing the package does not load the
library; the first call does, and fails loudly if it has not been built.
"""
from . import synth  # noqa: F401
from .binding import BFQ_BF16, BFQ_F32, BfqError, GemmOperand, Plan, backward_noalloc, lib, measure_fma_rates, measure_mma_rates  # noqa: F401
from .host_pipeline import HostForwardQuant  # noqa: F401
