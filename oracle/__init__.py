"""CPU oracle (test infrastructure only).

Plain C implementation of the memory-free bidirectional top_K step, loaded
through ctypes.  Nothing in the CUDA library imports or links this package;
only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
"""
from .ref import (build, ref_topk, ref_topk_rows, ref_aggregate, ref_step, StepResult,  # noqa: F401
                  ref_step_ef, EfResult, ref_lost_energy, ref_rho)
