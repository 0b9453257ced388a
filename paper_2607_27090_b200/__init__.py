"""B200-native retrieve + Chunked-RoPE KV injection (C-ABI library ``libmemstore.so`` plus a thin binding).

``from paper_2607_27090_b200 import MemStore`` loads the CUDA library on first use and raises if it has not
been built; there is no CPU fallback.  ``synth`` (seeded input generators) can be imported on its own.
"""


def __getattr__(name):
    if name in ("MemStore", "PagedCache", "MemStoreError", "memstore"):
        from . import memstore as _m

        return _m if name == "memstore" else getattr(_m, name)
    raise AttributeError(name)
