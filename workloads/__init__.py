"""Seeded synthetic workloads shared by the tests, the benchmark and the smoke check.

This package only produces input tensors (and names their shapes).  It holds
none of the convolution's arithmetic and is imported neither by the oracle nor
by the CUDA library.
"""
from .generate import (  # noqa: F401
    CONFIGS, ConvShape, make_inputs, uniform, normal, relu_normal, small_integers,
)
