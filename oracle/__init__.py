"""CPU oracle of the Sparsely-Gated Mixture-of-Experts layer.

TEST INFRASTRUCTURE. Nothing here is part of the product: only the tests, the
smoke check and the benchmark's CPU-baseline leg may import this package. It
shares no code with the CUDA library and imports nothing from it.

`moe_oracle` holds the method (numpy, float64 unless a passage fixes the
precision); `chain.c` holds the two single-precision steps whose rounding
order is fixed because they decide the routing.
"""
from . import moe_oracle  # noqa: F401
from .moe_oracle import build_chain_library  # noqa: F401
