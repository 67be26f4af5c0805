"""B200-native ROBE-Z embedding lookup (arXiv 2108.02191): a C-ABI CUDA library
(``librobe.so``, declared in ``include/robe.h``) and a thin binding of it.

The binding (and with it the shared library) is loaded at the first use of one of its
names, so that the seeded input generators in ``synth`` can be imported by a process that
never touches the CUDA library (the CPU-oracle timing arm of the benchmark).  There is no
fallback: if ``librobe.so`` is missing, that first use raises ImportError."""
import importlib

_SUBMODULES = ("binding", "synth", "build", "dp")


def __getattr__(name):
    if name in _SUBMODULES:
        return importlib.import_module("." + name, __name__)
    if name.startswith("__"):
        raise AttributeError(name)
    binding = importlib.import_module(".binding", __name__)
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
