"""Composed subkernels on B200: a module is an operator sequence, a decomposition splits it into
submodules with fixed contracts, one sm_100a subkernel is bound per submodule, and the composed
forward runs them on a CUDA stream.  The product is libmk.so (see include/mk.h); this package
holds its sources (csrc/), the in-tree build and a ctypes binding."""
from . import binding  # noqa: F401  (raises if libmk.so has not been built)
from .binding import Context, MkError, Module  # noqa: F401
