"""B200 (sm_100a) implementation of Draco's parameter-server hot path
(arXiv 1803.09877): redundant-gradient encoding, adversary location and exact
decoding for the repetition and cyclic codes.

The work is done by hand-written CUDA kernels behind a C ABI (``include/draco.h``,
``libdraco.so``); this package is a thin ctypes binding with the same names.
There is no CPU fallback: the first use of any name below loads ``libdraco.so``
and raises if it has not been built (``python -m paper_1803_09877_b200.build``).
The ``build`` submodule itself imports without the library.
"""
_BINDING_NAMES = ("ADV_CONST", "ADV_GAUSS", "ADV_REVGRAD", "CYC", "CYC_PACKED", "REP", "DracoError", "DracoInfo", "Plan",
                  "cyc_project_noalloc", "generate", "lib", "library_path")
__all__ = list(_BINDING_NAMES) + ["binding", "build", "sharding"]


def __getattr__(name):
    if name in _BINDING_NAMES or name == "binding":
        import importlib
        binding = importlib.import_module(".binding", __name__)
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
