"""B200-native decode attention over a head-mixed KV cache (full heads + sink/ring heads).

The product is ``librlkv.so`` (CUDA, sm_100a; C ABI in ``include/rlkv.h``); this package is its
thin ctypes binding.  ``paper_2510_08525_b200.binding`` loads the library and raises ImportError if
it has not been built -- there is no CPU or PyTorch fallback.  The binding is loaded on first use
of any of its names through the package, so that ``python -m paper_2510_08525_b200.build`` can
run before the library exists.
"""
import importlib

_SUBMODULES = ("binding", "build", "harness")


def __getattr__(name):
    if name in _SUBMODULES:
        return importlib.import_module(f"{__name__}.{name}")
    binding = importlib.import_module(f"{__name__}.binding")   # ImportError if librlkv.so is missing
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
