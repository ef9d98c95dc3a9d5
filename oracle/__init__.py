"""CPU oracle for the BWLA W1AX linear layer (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  The CUDA library and its Python binding never do.
"""
from .bwla_oracle import *  # noqa: F401,F403
