"""Reference oracle for the unit-scaled linear / FFN block (test infrastructure).

Plain, slow, fp64 NumPy restatement of what the unit-scaled ops compute, written
from the paper's definitions.  It exists only so that tests, the smoke check and
the benchmark's CPU-baseline leg have something independent to compare the CUDA
library with.  It shares no code with the CUDA path and the product never
imports it.
"""
