"""CPU oracle of the MoE-FFN layer.  Test infrastructure: only tests/, the smoke check and
bench.py's CPU-baseline / reference legs may import this package; the CUDA path never does."""
from .moe_oracle import (build_oracle, bwd, fwd, layout, route, swiglu_add, threads)  # noqa: F401
