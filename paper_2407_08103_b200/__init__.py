"""libcstr: regular-language constraints for batched LM decoding on one B200.

``cstr`` is the ctypes binding of the C ABI declared in ``include/cstr.h``;
``build`` compiles the CUDA sources in ``csrc/`` into ``libcstr.so`` in-tree.
"""

from . import build, cstr  # noqa: F401
from .cstr import *  # noqa: F401,F403
