"""Seeded synthetic inputs for the Draco encode / locate / decode path.

This package only *draws inputs*: per-partition gradients, the locator's random
projection vector, synthetic received matrices and adversarial corruptions.
It contains none of the method's arithmetic (no encoding, voting, locating or
decoding) and is the one module shared by the CPU oracle's tests and by the
CUDA path's tests and benchmark.  Everything is a pure function of
``(seed, row, coordinate)`` so any slice or scattered sample of a very large
input can be produced on its own.
"""
from .generator import (  # noqa: F401
    ADV_REVGRAD,
    ADV_CONST,
    ADV_GAUSS,
    INV_SIGMA_F32,
    IH_CENTER,
    splitmix64_at,
    row_key,
    approx_normal_at,
    approx_normal_rows,
    gradient_rows,
    projection_vector,
    complex_rows,
    choose_adversaries,
    apply_adversaries,
)
