"""DES-LOC fused optimizer step for NVIDIA B200: Python names for the C ABI of libdesloc.so.

``desloc_create / desloc_step / desloc_destroy`` and friends mirror include/desloc.h one to
one (see binding.py).  ``DesLoc`` is a small convenience wrapper that keeps torch tensors
alive and marshals their addresses; torch is used for device memory and streams only.

The shared library is loaded on first use of any of those names, so that
``paper_2505_22549_b200.build`` can be imported to (re)build it.  There is no fallback: if
the library is missing or lacks a symbol, that first use raises.
"""
import importlib

_LAZY_MODULES = ("binding", "module")


def __getattr__(name):
    if name in ("build", "dist"):
        return importlib.import_module(f"{__name__}.{name}")
    for mod in _LAZY_MODULES:
        m = importlib.import_module(f"{__name__}.{mod}")
        if hasattr(m, name):
            return getattr(m, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")


def load():
    """Load libdesloc.so now (raises if it is missing or stale) and return the ctypes handle."""
    return importlib.import_module(f"{__name__}.binding").raw_lib()
