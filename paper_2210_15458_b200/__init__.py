"""B200-native arithmetic-sampling decode (arXiv 2210.15458): thin Python binding over
the C-ABI CUDA library.  Importing the package does not load the library; the first
call of a bound function does, and fails loudly if it is missing."""
from . import synth  # noqa: F401  (seeded synthetic inputs; no CUDA needed)

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
