"""B200 (sm_100a) allowed-token mask build + apply for operator-automaton structured decoding.

The product is the C-ABI library ``libwg.so`` (``include/wg.h``); this package is its thin
Python binding.  Build the library with ``python -m paper_2507_16768_b200.build``.  The
binding is loaded on first use and raises ImportError if the library has not been built:
there is no CPU fallback.
"""
import importlib

__all__ = ["build", "binding"]


def __getattr__(name):
    if name == "build":
        return importlib.import_module(".build", __name__)
    binding = importlib.import_module(".binding", __name__)
    if name == "binding":
        return binding
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
