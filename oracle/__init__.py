"""CPU oracle of the RPS synchronisation step: TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the CUDA package and shares no code with it.
"""
from .rps_oracle import (  # noqa: F401
    ASSIGN_FIXED,
    ASSIGN_PERM,
    alpha_mc,
    bf16_to_double,
    block_size,
    build,
    diag,
    double_to_bf16,
    masks,
    noise,
    philox4x32,
    philox4x32_10,
    run,
    step,
    step_columns,
)
