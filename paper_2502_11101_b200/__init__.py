"""CacheFocus query-time path for B200: a ctypes binding over the C ABI in include/cachefocus.h.

Importing the package does not load the CUDA library; the first call does, and fails loudly if
the library has not been built (there is no CPU fallback)."""
from .binding import *  # noqa: F401,F403
