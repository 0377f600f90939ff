"""B200-native per-stage training library (C ABI in include/ftpipe.h) and its thin Python binding.

The binding (and with it the shared library) is loaded on first use, so that
`python -m paper_2110_02781_b200.build` can run before the library exists or after its ABI changed.
"""
import importlib


def __getattr__(name):
    if name in ("build", "replicas"):                      # plain submodules: never need the library
        return importlib.import_module("." + name, __name__)
    ft = importlib.import_module(".ftpipe", __name__)      # raises if libftpipe.so is missing: there is no fallback
    try:
        return getattr(ft, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
