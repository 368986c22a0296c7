"""CPU oracle for the R-FAST activation step: TEST INFRASTRUCTURE ONLY.

A plain, slow, event-driven fp64 implementation of Algorithm 1 (local view)
driven round by round as in Algorithm 2 (global view), plus plain per-node
gradient definitions.  It shares no code with the CUDA library and must never be
imported by it; only the tests, the smoke check and the benchmark's CPU-baseline
leg may use it.
"""

from .rfast_oracle import RFastOracle, run_schedule, rel_l2, from_workload
from .models import make_model, bf16_round

__all__ = ["RFastOracle", "run_schedule", "rel_l2", "from_workload", "make_model", "bf16_round"]
