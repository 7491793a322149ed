"""B200 (sm_100a) implementation of the HIGGS quantized linear layer.

The product is the CUDA shared library built from ``csrc/`` behind the C ABI of
``include/higgs.h``; this package is its ctypes binding (``binding.py``), whose
names are re-exported here on first use.  Using any of them fails loudly when the
library has not been built (``python -m paper_2411_17525_b200.build``): there is
no fallback path.
"""
import importlib

_BINDING = None


def __getattr__(name):
    global _BINDING
    if name.startswith("__"):
        raise AttributeError(name)
    if _BINDING is None:
        _BINDING = importlib.import_module(".binding", __name__)
    try:
        return getattr(_BINDING, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
