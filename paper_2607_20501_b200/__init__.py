"""Composed subkernels on B200: a module is an operator sequence, a decomposition splits it into
submodules with fixed contracts, one sm_100a subkernel is bound per submodule, and the composed
forward runs them on a CUDA stream.  The product is libmk.so (see include/mk.h); this package
holds its sources (csrc/), the in-tree build (build.py) and a ctypes binding (binding.py).

The binding is loaded on first use so that `python -m paper_2607_20501_b200.build` can run before
the library exists; using it without a built library raises (there is no fallback path)."""

_LAZY = {"Context", "MkError", "Module"}


def __getattr__(name):
    if name in _LAZY:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
