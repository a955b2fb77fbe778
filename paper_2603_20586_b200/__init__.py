"""B200 (sm_100a) FastMKA attention library: Python binding of the C ABI in ``include/mka.h``.

The package holds the CUDA sources (``csrc/``), the build step (``build.py``) and the ctypes binding
(``binding.py``).  Attributes are resolved lazily from the binding so that
``python -m paper_2603_20586_b200.build`` can run before the library exists; the first use of any
entry point loads ``libmka_b200.so`` and raises if it is missing or stale.  There is no CPU or
PyTorch fallback.
"""
import importlib

_BINDING = None


def __getattr__(name):
    global _BINDING
    if name == "build":
        return importlib.import_module(".build", __name__)
    if _BINDING is None:
        _BINDING = importlib.import_module(".binding", __name__)
    if name == "binding":
        return _BINDING
    try:
        return getattr(_BINDING, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
