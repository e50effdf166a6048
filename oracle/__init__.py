"""fp64 CPU oracle of the GELO obfuscated Q/K/V offload -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never imports it.
"""
from .oracle import *  # noqa: F401,F403
