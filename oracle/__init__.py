"""CPU oracle for the forward convolution -- test infrastructure only.

Nothing in the product package may import this.  Allowed callers: the tests,
the smoke check and the benchmark's cpu-baseline / reference legs.
"""
from .conv2d_oracle import build, conv2d_oracle, conv2d_oracle_range, oracle_threads  # noqa: F401
