"""CPU oracle of the planner hot path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.
"""
from .hap_oracle import *  # noqa: F401,F403
