"""CPU fp64 oracle for the L4Q linear layer (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA product path never does.
"""
from .l4q_oracle import (  # noqa: F401
    L4QSpec,
    grid_bounds,
    merge,
    prequant,
    quant_codes,
    dequant,
    fake_quant_weight,
    forward,
    backward,
    pack_int,
    unpack_int,
    round_to_bf16,
)
