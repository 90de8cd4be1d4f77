"""B200-native batched evaluation of DiSCo's dispatch and migration policy (arXiv 2502.11417).

`api` binds the C ABI of libdisco.so (hand-written CUDA, sm_100a); `synth` draws the seeded workloads.
"""
from . import synth  # noqa: F401
from .api import (  # noqa: F401
    Trace, DiscoError, lib, library_path, policy_array, NBINS, SERVER_ONLY, DEVICE_ONLY, RACE, EINFEASIBLE,
)
