"""CPU oracle for the LampAttention forward pass (test infrastructure only).

Nothing in the product package imports this; only tests, the smoke check and the
benchmark's CPU-baseline leg do.
"""
from .lamp_oracle import (  # noqa: F401
    COMPACT_BRANCH, FORCE_16BIT, H16_SEQ, SR_E4M3, FORCE_8BIT, NO_STAGE1, OracleResult, build, lib, run_units, run_all, rne_e4m3_array, exp16_array,
)
