"""CPU oracle of the MoE-FFN layer.  Test infrastructure: only tests/, the smoke check and
bench.py's CPU-baseline / reference legs may import this package; the CUDA path never does."""
from .moe_oracle import (build_oracle, bwd, fwd, layout, route, router_bwd, router_fwd, router_logits,  # noqa: F401
                         swiglu_add, threads)  # noqa: F401
