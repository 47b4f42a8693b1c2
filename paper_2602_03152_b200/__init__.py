"""B200 (sm_100a) decode-time hot path of FASA (arxiv 2602.03152).

`synth` draws seeded inputs; `binding` wraps the C-ABI CUDA library
(`libfasa.so`, built by `build.py`) and raises if it is missing.  Importing
the package loads neither: each is imported on first attribute access.
"""
import importlib

__all__ = ["synth", "binding", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
