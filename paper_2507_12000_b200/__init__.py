"""B200 (sm_100a) library for the verification round of Distributed Split Speculative Decoding.

`paper_2507_12000_b200.binding` holds the Python front end of the C-ABI library libdssd.so;
`paper_2507_12000_b200.build` compiles it.  Other attribute access on the package forwards to
the binding, which raises ImportError when the library has not been built: there is no CPU path.
"""
import importlib

_SUBMODULES = ("binding", "build")


def __getattr__(name):
    if name.startswith("__"):
        raise AttributeError(name)
    if name in _SUBMODULES:
        return importlib.import_module(f"{__name__}.{name}")
    return getattr(importlib.import_module(f"{__name__}.binding"), name)
