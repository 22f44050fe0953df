"""Per-example gradient statistics for linear layers on B200 (sm_100a).

``pe_linear_stats``, ``pe_token_sqstats``, ``microadam_step`` and ``microsignsgd_step`` are
thin wrappers over the C-ABI library built from ``csrc/``; every step runs in its CUDA kernels.
``inputs`` holds the seeded synthetic input generators.
"""
from . import inputs  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import __all__ as _binding_all

__all__ = ["inputs"] + list(_binding_all)
