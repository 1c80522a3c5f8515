"""CPU oracle for the DistSim timeline engine -- TEST INFRASTRUCTURE ONLY.

A ctypes wrapper around ``distsim_oracle.c`` (plain C, single-threaded).  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA engine never does, and this package imports nothing from it.
"""
from .oracle import (  # noqa: F401
    KINDS, Candidate, OracleError, SimResult, build, count, enumerate_at, eval_indices,
    eval_indices_parallel, ring_allreduce_ns, allreduce_ns, all_to_all_ns, p2p_ns, simulate,
)
