"""CPU oracle of the SAT partition-parallel GCN step.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never imports it.
"""
from .build import build_oracle, oracle_lib_path  # noqa: F401
