"""B200 (sm_100a) implementation of the ESP decode-and-verify step.

The product is the C-ABI library ``libesp_b200.so`` (declared in
``include/esp.h``); this package is its thin ctypes binding.  Importing it
never falls back to a CPU path: without the compiled library every call
raises.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
