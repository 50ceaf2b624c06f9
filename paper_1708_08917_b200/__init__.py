"""Block-circulant layer forward pass on B200 (sm_100a) behind a C ABI.

``binding`` mirrors ``include/circ.h`` one to one (ctypes, marshalling only); ``synth`` draws the
seeded benchmark inputs; ``build`` compiles ``libcirc.so`` in-tree.  Nothing is computed in Python.
"""
from .binding import *  # noqa: F401,F403
from .binding import CircError, load  # noqa: F401
