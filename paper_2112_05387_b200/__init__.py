"""Layer-parallel training step on one B200: Python binding over the C-ABI library (include/lp.h).

The binding only marshals arguments; every step of the path runs in the CUDA kernels of
``liblp.so``.  Importing this package does not load the library; the first call does, and raises
if the library has not been built (``python -c 'import __graft_entry__ as g; g.build()'``).
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
