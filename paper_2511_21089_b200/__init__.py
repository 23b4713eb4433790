"""B200-native MLPMoE forward path (arXiv 2511.21089): Python binding over the C-ABI library.

`synth` (seeded input generators) is importable without the CUDA library; every
compute entry point lives in `binding` and raises if the library is missing.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
