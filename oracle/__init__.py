"""CPU oracle (test infrastructure): see cachefocus_oracle.py."""
from .cachefocus_oracle import *  # noqa: F401,F403
from .cachefocus_oracle import (ALLOC_ALIGN, ALLOC_NONE, ALLOC_SORT, ROPE_HALF, ROPE_INTERLEAVED,
                                RangeError)  # noqa: F401
