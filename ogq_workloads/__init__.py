"""Seeded synthetic gradient buckets.

This module holds no quantization arithmetic.  It only produces the inputs
(tensor shapes, offsets and fp32 values) that both the CPU oracle's tests and
the CUDA path's tests and benchmark consume, so that the two sides always see
the same numbers.  All draws come from ``numpy.random.Generator(PCG64(seed))``.

Scale conventions: a Gaussian "N(0, x)" has standard deviation x, a Laplace
"Laplace(0, x)" has scale parameter b = x, and "Student-t(nu) scaled by x" is
x times a standard t variate.
"""
from .shapes import resnet50_shapes, vgg19_shapes, numel
from .buckets import (
    Bucket,
    laplace,
    gaussian,
    student_t,
    mixture,
    config1,
    config2,
    resnet50_bucket,
    vgg19_bucket,
    sweep_tensor,
    offsets_from_sizes,
)

__all__ = [
    "resnet50_shapes",
    "vgg19_shapes",
    "numel",
    "Bucket",
    "laplace",
    "gaussian",
    "student_t",
    "mixture",
    "config1",
    "config2",
    "resnet50_bucket",
    "vgg19_bucket",
    "sweep_tensor",
    "offsets_from_sizes",
]
