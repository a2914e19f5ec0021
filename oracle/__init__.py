"""Float64 CPU oracle for the DPPO per-token loss path.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain restatement of the
paper's definitions that the CUDA library is checked against.  It shares no
code with the CUDA path and must never be imported by the product package:
only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
use it.
"""
