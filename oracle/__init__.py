"""CPU oracle of the DiSCo policy evaluation -- TEST INFRASTRUCTURE ONLY.

Only the test suite, the smoke check and the benchmark's CPU-baseline leg may
import this package.  The CUDA library never does, and shares nothing with it.
"""
from .binding import (  # noqa: F401
    Oracle, OracleStats, build_oracle, lib, server_struct, device_struct, policy_struct,
    NBINS, SERVER_ONLY, DEVICE_ONLY, RACE,
)
