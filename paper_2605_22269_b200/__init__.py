"""MuKV compression + retrieval hot path for NVIDIA B200 (sm_100a).

``binding`` wraps the C ABI declared in ``include/mukv.h`` (same names, argument
marshalling only); ``synth`` holds the seeded input generators.
"""
from .binding import (MukvConfig, MukvContext, MukvError, MukvStats, load_library,  # noqa: F401
                      BF16, FP32, RETR_PARALLEL, RETR_HIER, RETR_SEMI)
