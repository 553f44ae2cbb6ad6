"""B200-native decode attention over a head-mixed KV cache (full heads + sink/ring heads).

The product is ``librlkv.so`` (CUDA, sm_100a; C ABI in ``include/rlkv.h``); this package is its
thin ctypes binding.  ``from paper_2510_08525_b200 import binding`` loads the library and raises if
it has not been built -- there is no CPU or PyTorch fallback.
"""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403
