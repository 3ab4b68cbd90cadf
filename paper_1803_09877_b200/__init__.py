"""B200 (sm_100a) implementation of Draco's parameter-server hot path
(arXiv 1803.09877): redundant-gradient encoding, adversary location and exact
decoding for the repetition and cyclic codes.

The work is done by hand-written CUDA kernels behind a C ABI (``include/draco.h``,
``libdraco.so``); this package is a thin ctypes binding with the same names.
There is no CPU fallback: a missing library raises at import of ``binding``.
"""
from .binding import (  # noqa: F401
    ADV_CONST,
    ADV_GAUSS,
    ADV_REVGRAD,
    CYC,
    REP,
    DracoError,
    DracoInfo,
    Plan,
    cyc_project_noalloc,
    generate,
    lib,
    library_path,
)
