"""One routed MoE decode layer on VQ + shared-basis low-rank expert weights, for sm_100a.

``synth`` (seeded inputs) imports without the CUDA library; everything else needs the built
shared library and fails loudly when it is missing.
"""

__all__ = ["synth", "binding", "accounting", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
