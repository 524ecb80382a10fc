"""CPU oracle of the batched WWW.Serve network step: test infrastructure only.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package.  It never imports the CUDA package.
"""
from .binding import Oracle, build, lib, STAT_NAMES, TABLES  # noqa: F401
