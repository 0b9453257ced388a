"""B200-native retrieve + Chunked-RoPE KV injection (C-ABI library ``libmemstore.so`` plus a thin binding).

``from paper_2607_27090_b200 import MemStore`` loads the binding; creating a store loads the CUDA library
and raises if it has not been built.  There is no CPU fallback.  ``synth`` (seeded input generators) can
be imported on its own.
"""
import importlib

_BINDING_NAMES = ("MemStore", "PagedCache", "MemStoreError")


def __getattr__(name):
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(".memstore", __name__), name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
