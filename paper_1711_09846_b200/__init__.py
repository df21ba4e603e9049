"""Lockstep Population Based Training on one B200: CUDA library + thin ctypes binding."""
from .binding import (EXPORTS, energy_fitness_static, grouped_gemm, selftest_bounded_wait, PbtError, Population, library_path, load_library, param_count,  # noqa: F401
                      spec_from_config)
