"""B200-native dual-state linear attention (DSLA) layer: prefill and decode.

The compute lives in ``libdsla.so`` (hand-written sm_100a CUDA behind a C ABI,
declared in ``include/dsla.h``).  ``binding`` marshals arguments only.  There is
no CPU fallback: importing ``binding`` (or any name re-exported from it) raises
if the shared library has not been built.
"""
import importlib

__all__ = ["binding", "inputs", "build"]


def __getattr__(name):
    if name in ("binding", "inputs", "build"):
        return importlib.import_module(f"{__name__}.{name}")
    b = importlib.import_module(f"{__name__}.binding")
    try:
        return getattr(b, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
