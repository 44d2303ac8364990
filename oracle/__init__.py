"""CPU oracle (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It never imports the CUDA library or its Python binding.
"""
from .oracle import *  # noqa: F401,F403
