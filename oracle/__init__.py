"""CPU oracle for block-sparse fused attention: test infrastructure, not product code.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA path and never imports it.
"""
from .steel_oracle import (  # noqa: F401
    OracleProblem, build, rows, alg1_blocks, classify, count_tiles, allowed, max_threads,
)
