"""Thin Python binding of ``libmemstore.so`` (argument marshalling only).

Every step of the path (scoring, top-k, fact resolution, position assignment, slot mapping, RoPE, the
K/V scatter) runs in the CUDA kernels behind the C ABI of ``include/memstore.h``; this module converts
torch tensors to raw device pointers and checks dtypes and shapes.  torch is used for device memory and
streams only.  If the library has not been built, creating a MemStore raises: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libmemstore.so"

MS_OK = 0
STATUS_NAMES = {0: "MS_OK", 1: "MS_ERR_INVALID_ARG", 2: "MS_ERR_UNSUPPORTED", 3: "MS_ERR_OOM", 4: "MS_ERR_CAPACITY", 5: "MS_ERR_CUDA"}
REQ_BAD_FACT_ID, REQ_NOT_RESIDENT, REQ_BLOCK_TABLE_SHORT, REQ_BAD_BLOCK_ID, REQ_POSITION_OVERFLOW = 1, 2, 4, 8, 16
DTYPE_F32, DTYPE_F16, DTYPE_BF16 = 0, 1, 2
ROPE_HALF_SPLIT, ROPE_INTERLEAVED = 0, 1
INJECT_REVERSE = 1
INJECT_PREFIX = 2
RETRIEVE_ANN = 4
INPUTS_STABLE = 8
SERVE_EARLY_RETURN = 16
COMPOSE_CACHE_ALL = 1
CACHE_BF16, CACHE_FP8_E4M3 = 0, 1
STORE_TMA_COPY_PATH = 1
REQ_KERNEL_TIMEOUT = 32
REQ_BAD_START = 64


class MemStoreError(RuntimeError):
    def __init__(self, code: int, msg: str = ""):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {msg}")
        self.code = code


class _Config(C.Structure):
    _fields_ = [
        ("device", C.c_int32), ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("kv_dtype", C.c_int32), ("emb_dim", C.c_int32), ("emb_dtype", C.c_int32), ("rope_style", C.c_int32),
        ("rope_theta", C.c_double), ("inv_freq_override", C.POINTER(C.c_float)), ("max_position", C.c_int64),
        ("n_users", C.c_int32), ("flags", C.c_uint32), ("max_facts_per_user", C.c_int64),
        ("max_kv_tokens", C.c_int64), ("kv_arena", C.c_void_p), ("kv_arena_bytes", C.c_size_t),
        ("max_host_kv_tokens", C.c_int64), ("rotary_dim", C.c_int32), ("reserved1", C.c_int32),
    ]  # fmt: skip


class _PagedCache(C.Structure):
    _fields_ = [
        ("k_base", C.c_void_p), ("v_base", C.c_void_p), ("layer_stride", C.c_int64), ("block_stride", C.c_int64),
        ("token_stride", C.c_int64), ("head_stride", C.c_int64), ("num_blocks", C.c_int64),
        ("block_size", C.c_int32), ("dtype", C.c_int32), ("k_scale", C.c_float), ("v_scale", C.c_float),
    ]  # fmt: skip


class _AnnParams(C.Structure):
    _fields_ = [("beam", C.c_int32), ("parents", C.c_int32), ("n_entry", C.c_int32), ("max_iters", C.c_int32)]


class _Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "n_facts", "n_resident_facts", "kv_tokens_used", "retrieve_calls", "inject_calls", "kernels_launched",
        "arena_bytes", "embedding_bytes", "host_kv_tokens_used", "kernel_timeouts", "filter_fixups", "n_removed_facts", "compose_cache_hits", "compose_cache_fills", "compose_cache_segments", "filter_fixup_overflows", "filter_list_queries", "filter_list_rows", "filter_list_fallbacks")]  # fmt: skip


# every symbol include/memstore.h declares
EXPORTS = (
    "memstore_version", "memstore_arena_bytes", "memstore_create", "memstore_destroy", "memstore_add_fact",
    "memstore_add_facts", "memstore_retrieve", "memstore_inject", "memstore_stats", "memstore_last_error",
    "memstore_set_profile_events", "memstore_set_profile_repeats", "memstore_retrieve_static", "memstore_serve_host",
    "memstore_retrieve_inject", "memstore_add_facts_host", "memstore_set_prefix", "memstore_rope_table_llama3",
    "memstore_build_graph", "memstore_set_graph", "memstore_get_graph", "memstore_retrieve_ann", "memstore_graph_append",
    "memstore_test_hooks", "memstore_reserve", "memstore_compose_cache", "memstore_remove_fact", "memstore_set_graph_user",
    "memstore_get_graph_user", "memstore_retrieve_ann_users",
)  # fmt: skip

_lib = None


def load_library() -> C.CDLL:
    """dlopen the in-tree CUDA library; raises if it is missing (build it with ``__graft_entry__.build()``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise ImportError(
            f"{_LIB_PATH} not found: build it with `python -m paper_2607_27090_b200.build` "
            "(nvcc, sm_100a). This package has no CPU fallback."
        )
    L = C.CDLL(str(_LIB_PATH))
    vp, i32, i64, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32
    L.memstore_version.restype = C.c_char_p
    L.memstore_version.argtypes = []
    L.memstore_arena_bytes.restype = C.c_size_t
    L.memstore_arena_bytes.argtypes = [C.POINTER(_Config)]
    L.memstore_create.restype = i32
    L.memstore_create.argtypes = [C.POINTER(_Config), C.POINTER(vp)]
    L.memstore_destroy.restype = i32
    L.memstore_destroy.argtypes = [vp]
    L.memstore_add_fact.restype = i32
    L.memstore_add_fact.argtypes = [vp, i32, vp, vp, vp, i32, C.POINTER(i32), vp]
    L.memstore_add_facts.restype = i32
    L.memstore_add_facts.argtypes = [vp, i32, i64, vp, vp, vp, C.POINTER(i32), C.POINTER(i32), vp]
    L.memstore_add_facts_host.restype = i32
    L.memstore_add_facts_host.argtypes = [vp, i32, i64, vp, vp, vp, C.POINTER(i32), C.POINTER(i32), vp]
    L.memstore_retrieve.restype = i32
    L.memstore_build_graph.restype = i32
    L.memstore_build_graph.argtypes = [vp, i32, vp]
    L.memstore_graph_append.restype = i32
    L.memstore_graph_append.argtypes = [vp, vp]
    L.memstore_compose_cache.restype = i32
    L.memstore_compose_cache.argtypes = [vp, C.c_size_t, C.c_int32, C.c_uint32]
    L.memstore_reserve.restype = i32
    L.memstore_reserve.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_int32]
    L.memstore_test_hooks.restype = i32
    L.memstore_test_hooks.argtypes = [vp, C.c_uint32, C.c_int32]
    L.memstore_set_graph.restype = i32
    L.memstore_set_graph.argtypes = [vp, vp, i64, i32, vp]
    L.memstore_get_graph.restype = i32
    L.memstore_get_graph.argtypes = [vp, vp, i64, C.POINTER(i64), C.POINTER(i32), vp]
    L.memstore_retrieve_ann.restype = i32
    L.memstore_retrieve_ann.argtypes = [vp, vp, i32, i32, C.POINTER(_AnnParams), vp, vp, vp, vp]
    L.memstore_retrieve_ann_users.restype = i32
    L.memstore_retrieve_ann_users.argtypes = [vp, vp, vp, i32, i32, C.POINTER(_AnnParams), vp, vp, vp, vp]
    L.memstore_set_graph_user.restype = i32
    L.memstore_set_graph_user.argtypes = [vp, i32, vp, i64, i32, vp]
    L.memstore_get_graph_user.restype = i32
    L.memstore_get_graph_user.argtypes = [vp, i32, vp, i64, C.POINTER(i64), C.POINTER(i32), vp]
    L.memstore_remove_fact.restype = i32
    L.memstore_remove_fact.argtypes = [vp, i32, vp]
    L.memstore_rope_table_llama3.restype = i32
    L.memstore_rope_table_llama3.argtypes = [i32, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, C.POINTER(C.c_float)]
    L.memstore_set_prefix.restype = i32
    L.memstore_set_prefix.argtypes = [vp, vp, vp, i32, vp]
    L.memstore_retrieve.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
    L.memstore_retrieve_static.restype = i32
    L.memstore_retrieve_static.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
    L.memstore_retrieve_inject.restype = i32
    L.memstore_retrieve_inject.argtypes = [vp, vp, vp, i32, i32, vp, vp, i32, C.POINTER(_PagedCache), vp, vp, vp, vp, vp, i64, u32, vp]
    L.memstore_serve_host.restype = i32
    L.memstore_serve_host.argtypes = [vp, vp, i32, i32, i32, vp, i32, C.POINTER(_PagedCache), u32, vp, vp, vp, vp]
    L.memstore_inject.restype = i32
    L.memstore_inject.argtypes = [vp, vp, i32, i32, vp, vp, i32, C.POINTER(_PagedCache), vp, vp, vp, i64, u32, vp]
    L.memstore_stats.restype = i32
    L.memstore_stats.argtypes = [vp, C.POINTER(_Stats)]
    L.memstore_set_profile_events.restype = i32
    L.memstore_set_profile_events.argtypes = [vp, vp, vp]
    L.memstore_set_profile_repeats.restype = i32
    L.memstore_set_profile_repeats.argtypes = [vp, i32]
    L.memstore_last_error.restype = C.c_char_p
    L.memstore_last_error.argtypes = [vp]
    _lib = L
    return L


def _dev_ptr(t: torch.Tensor | None, dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream_ptr(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def rope_table_llama3(rotary_dim, rope_theta, factor=8.0, low_freq_factor=1.0, high_freq_factor=4.0, original_max_position=8192):
    """The Llama-3.1 family's rescaled frequency table (computed by the library) as a list of floats for
    ``MemStore(inv_freq_override=...)``."""
    out = (C.c_float * (rotary_dim // 2))()
    rc = load_library().memstore_rope_table_llama3(rotary_dim, float(rope_theta), float(factor), float(low_freq_factor),
                                                   float(high_freq_factor), float(original_max_position), out)  # fmt: skip
    if rc != MS_OK:
        raise MemStoreError(rc, "memstore_rope_table_llama3")
    return list(out)


@dataclass
class PagedCache:
    """A caller-owned paged KV cache: two bf16 tensors and strides in elements (see ``ms_paged_cache``)."""

    k: torch.Tensor
    v: torch.Tensor
    layer_stride: int
    block_stride: int
    token_stride: int
    head_stride: int
    num_blocks: int
    block_size: int
    layout: str = "NHD"  # informational: how `allocate` shaped the tensors
    k_scale: float = 1.0  # 8-bit (uint8, e4m3 codes) caches only: the cache holds K / k_scale and V / v_scale
    v_scale: float = 1.0

    @classmethod
    def allocate(cls, n_layers, num_blocks, block_size, n_kv_heads, head_dim, device, layout="NHD", stacked=False, fill_bits=None,
                 fp8=False, k_scale=1.0, v_scale=1.0):  # fmt: skip
        """Allocate a cache. ``layout`` "NHD": [L][blocks][bs][h][d]; "HND": [L][blocks][h][bs][d].
        ``stacked``: K and V are planes 0 and 1 of one buffer [L][2][blocks]..., else separate buffers.
        ``fp8``: one byte per element (uint8 tensors of e4m3 codes) with the given per-tensor scales;
        ``fill_bits`` is then a byte."""
        shape = (num_blocks, block_size, n_kv_heads, head_dim) if layout == "NHD" else (num_blocks, n_kv_heads, block_size, head_dim)
        blk = block_size * n_kv_heads * head_dim
        dt = torch.uint8 if fp8 else torch.bfloat16
        if stacked:
            buf = torch.empty((n_layers, 2, *shape), dtype=dt, device=device)
            k, v = buf[:, 0], buf[:, 1]
            layer_stride = 2 * num_blocks * blk
            keep = buf
        else:
            k = torch.empty((n_layers, *shape), dtype=dt, device=device)
            v = torch.empty((n_layers, *shape), dtype=dt, device=device)
            layer_stride = num_blocks * blk
            keep = None
        if fill_bits is not None:
            for t in ((keep,) if stacked else (k, v)):
                if fp8:
                    t.fill_(fill_bits)
                else:
                    t.view(torch.int16).fill_(fill_bits - 0x10000 if fill_bits >= 0x8000 else fill_bits)
        token_stride, head_stride = (n_kv_heads * head_dim, head_dim) if layout == "NHD" else (head_dim, block_size * head_dim)
        c = cls(k, v, layer_stride, blk, token_stride, head_stride, num_blocks, block_size)
        c._keep = keep
        c.layout = layout
        c.k_scale, c.v_scale = float(k_scale), float(v_scale)
        return c

    @property
    def fp8(self) -> bool:
        return self.k.dtype == torch.uint8

    def _struct(self) -> _PagedCache:
        # (made once per state of the cache object: the calls of a serving loop pass the same cache every time)
        key = (self.k.data_ptr(), self.v.data_ptr(), self.layer_stride, self.block_stride, self.token_stride, self.head_stride,
               self.num_blocks, self.block_size, self.fp8, self.k_scale, self.v_scale)  # fmt: skip
        made = getattr(self, "_made", None)
        if made is not None and made[0] == key:
            return made[1]
        for t, n in ((self.k, "k"), (self.v, "v")):
            if not t.is_cuda or t.dtype not in (torch.bfloat16, torch.uint8) or t.dtype != self.k.dtype:
                raise TypeError(f"cache.{n} must be a CUDA bfloat16 (or, for an 8-bit cache, uint8) tensor")
        cs = _PagedCache(self.k.data_ptr(), self.v.data_ptr(), self.layer_stride, self.block_stride,
                         self.token_stride, self.head_stride, self.num_blocks, self.block_size,
                         CACHE_FP8_E4M3 if self.fp8 else CACHE_BF16, self.k_scale, self.v_scale)  # fmt: skip
        self._made = (key, cs)
        return cs


class MemStore:
    """Handle of one ``memstore_t`` (see ``include/memstore.h`` for the meaning of every argument)."""

    def __init__(self, *, device=0, n_layers, n_kv_heads, head_dim, emb_dim, emb_dtype=torch.float16, rope_theta=1.0e4,
                 rope_style=ROPE_HALF_SPLIT, inv_freq_override=None, max_position=1 << 24, n_users=1,
                 max_facts_per_user, max_kv_tokens, kv_arena: torch.Tensor | None = None, flags=0, max_host_kv_tokens=0,
                 rotary_dim=0):  # fmt: skip
        self._lib = load_library()
        self._h = C.c_void_p()
        self.device = torch.device("cuda", device if isinstance(device, int) else torch.device(device).index or 0)
        self.emb_torch_dtype = emb_dtype
        emb_code = {torch.float32: DTYPE_F32, torch.float16: DTYPE_F16}.get(emb_dtype)
        if emb_code is None:
            raise TypeError("emb_dtype must be torch.float32 or torch.float16")
        ov = None
        if inv_freq_override is not None:
            vals = [float(x) for x in inv_freq_override]
            ov = (C.c_float * len(vals))(*vals)
            if len(vals) != (rotary_dim or head_dim) // 2:
                raise ValueError("inv_freq_override needs rotary_dim/2 (head_dim/2) entries")
        self._arena = kv_arena
        cfg = _Config(self.device.index, n_layers, n_kv_heads, head_dim, DTYPE_BF16, emb_dim, emb_code, rope_style,
                      float(rope_theta), ov, max_position, n_users, flags, max_facts_per_user, max_kv_tokens,
                      kv_arena.data_ptr() if kv_arena is not None else None,
                      kv_arena.numel() * kv_arena.element_size() if kv_arena is not None else 0, max_host_kv_tokens,
                      rotary_dim, 0)  # fmt: skip
        self.n_layers, self.n_kv_heads, self.head_dim, self.emb_dim = n_layers, n_kv_heads, head_dim, emb_dim
        rc = self._lib.memstore_create(C.byref(cfg), C.byref(self._h))
        if rc != MS_OK:
            self._h = C.c_void_p()
            raise MemStoreError(rc, "memstore_create")

    # -- helpers ---------------------------------------------------------------------------------
    def _check(self, rc: int):
        if rc != MS_OK:
            raise MemStoreError(rc, self._lib.memstore_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.memstore_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # -- the four calls ---------------------------------------------------------------------------
    def add_fact(self, emb, k_pre=None, v=None, user=0, stream=None) -> int:
        n_tokens = 0 if k_pre is None else k_pre.shape[1]
        out = C.c_int32(-1)
        rc = self._lib.memstore_add_fact(self._h, user, _dev_ptr(emb, self.emb_torch_dtype, "emb"),
                                         _dev_ptr(k_pre, torch.bfloat16, "k_pre"), _dev_ptr(v, torch.bfloat16, "v"),
                                         n_tokens, C.byref(out), _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out.value

    def set_prefix(self, k_pre=None, v=None, stream=None) -> None:
        """The fixed instruction prefix placed before the facts by injections with ``INJECT_PREFIX``:
        ``k_pre``/``v`` [L, n, h, d] bf16 on the device (keys before RoPE); ``None`` removes it."""
        n_tokens = 0 if k_pre is None else k_pre.shape[1]
        rc = self._lib.memstore_set_prefix(self._h, _dev_ptr(k_pre, torch.bfloat16, "k_pre"), _dev_ptr(v, torch.bfloat16, "v"),
                                           n_tokens, _stream_ptr(stream))  # fmt: skip
        self._check(rc)

    def add_facts(self, embs, n_tokens, k_pre=None, v=None, user=0, stream=None) -> int:
        """``n_tokens``: host sequence of ints; ``k_pre``/``v``: [L, sum(n_tokens), h, d] bf16 on the device."""
        n = embs.shape[0]
        lens = (C.c_int32 * n)(*[int(x) for x in n_tokens])
        out = C.c_int32(-1)
        rc = self._lib.memstore_add_facts(self._h, user, n, _dev_ptr(embs, self.emb_torch_dtype, "embs"),
                                          _dev_ptr(k_pre, torch.bfloat16, "k_pre"), _dev_ptr(v, torch.bfloat16, "v"),
                                          lens, C.byref(out), _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out.value

    def add_facts_host(self, embs, n_tokens, k_pre_host, v_host, user=0, stream=None) -> int:
        """Like ``add_facts`` but K/V are HOST arrays (numpy uint16 bf16 bits or CPU bf16 tensors, [L, sum(n_tokens), h, d])
        that go to the store's pinned host arena; injection reads them over PCIe."""
        import numpy as np

        def host_ptr(a):
            if isinstance(a, torch.Tensor):
                assert not a.is_cuda and a.is_contiguous() and a.element_size() == 2
                return C.c_void_p(a.data_ptr())
            assert isinstance(a, np.ndarray) and a.flags.c_contiguous and a.itemsize == 2
            return C.c_void_p(a.ctypes.data)

        n = embs.shape[0]
        lens = (C.c_int32 * n)(*[int(x) for x in n_tokens])
        out = C.c_int32(-1)
        rc = self._lib.memstore_add_facts_host(self._h, user, n, _dev_ptr(embs, self.emb_torch_dtype, "embs"), host_ptr(k_pre_host),
                                               host_ptr(v_host), lens, C.byref(out), _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out.value

    def retrieve(self, queries, k, query_users=None, out_ids=None, out_scores=None, want_scores=True, stream=None):
        nq = queries.shape[0]
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
        if out_scores is None and want_scores:
            out_scores = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
        rc = self._lib.memstore_retrieve(self._h, _dev_ptr(queries, self.emb_torch_dtype, "queries"),
                                         _dev_ptr(query_users, torch.int32, "query_users"), nq, k,
                                         _dev_ptr(out_ids, torch.int32, "out_ids"),
                                         _dev_ptr(out_scores, torch.float32, "out_scores"), _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out_ids, out_scores

    # -- graph index ------------------------------------------------------------------------------
    def build_graph(self, degree=64, stream=None) -> None:
        """Exact neighbour graph of all facts present (single-segment stores), built on the device."""
        self._check(self._lib.memstore_build_graph(self._h, degree, _stream_ptr(stream)))

    def compose_cache(self, budget_bytes: int, max_tokens_per_segment: int = 0, cache_all: bool = False) -> None:
        """Keep composed segments of earlier requests in HBM (``budget_bytes`` = 0 switches the cache off)."""
        self._check(self._lib.memstore_compose_cache(self._h, int(budget_bytes), int(max_tokens_per_segment), COMPOSE_CACHE_ALL if cache_all else 0))

    def reserve(self, nq: int = 0, k: int = 0, nreq: int = 0, max_tokens_per_request: int = 0, max_blocks: int = 0) -> None:
        """Allocate every scratch buffer that calls of these sizes need, so that they allocate nothing later."""
        self._check(self._lib.memstore_reserve(self._h, nq, k, nreq, max_tokens_per_request, max_blocks))

    def test_hooks(self, wait_poll_limit: int = 0, mute_producers: bool = False) -> None:
        """Test aid: shorten every bounded wait of the staged kernels and silence their producer roles, so that the
        time-out reporting can be exercised; ``test_hooks()`` restores normal behaviour."""
        self._check(self._lib.memstore_test_hooks(self._h, int(wait_poll_limit), int(bool(mute_producers))))

    def graph_append(self, stream=None) -> None:
        """Grow the graph for the facts added since it was built, set or last grown."""
        self._check(self._lib.memstore_graph_append(self._h, _stream_ptr(stream)))

    def set_graph(self, graph: torch.Tensor, user: int = 0, stream=None) -> None:
        """Install the graph of ``user``'s segment: int32 device tensor [n_rows, degree] of rows of that segment."""
        self._check(self._lib.memstore_set_graph_user(self._h, user, _dev_ptr(graph, torch.int32, "graph"), graph.shape[0],
                                                      graph.shape[1], _stream_ptr(stream)))  # fmt: skip

    def get_graph(self, user: int = 0, stream=None) -> torch.Tensor:
        rows, deg = C.c_int64(0), C.c_int32(0)
        self._check(self._lib.memstore_get_graph_user(self._h, user, None, 0, C.byref(rows), C.byref(deg), _stream_ptr(stream)))
        out = torch.empty((rows.value, deg.value), dtype=torch.int32, device=self.device)
        self._check(self._lib.memstore_get_graph_user(self._h, user, _dev_ptr(out, torch.int32, "out"), out.numel(), None, None,
                                                      _stream_ptr(stream)))  # fmt: skip
        return out

    def remove_fact(self, fact_id: int, stream=None) -> None:
        """Take a fact out: retrieval never returns it again, injection refuses its id (MS_REQ_NOT_RESIDENT)."""
        self._check(self._lib.memstore_remove_fact(self._h, int(fact_id), _stream_ptr(stream)))

    def retrieve_ann(self, queries, k, beam=0, parents=0, n_entry=0, max_iters=0, out_ids=None, out_scores=None, want_scores=True,
                     want_counters=False, stream=None, query_users=None):  # fmt: skip
        """Beam search over the graph (0 = the library's default for that parameter).  Returns (ids, scores) or, with
        ``want_counters``, (ids, scores, counters [nq, 2] = steps taken and rows scored)."""
        nq = queries.shape[0]
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
        if out_scores is None and want_scores:
            out_scores = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
        counters = torch.zeros((nq, 2), dtype=torch.int32, device=queries.device) if want_counters else None
        prm = _AnnParams(beam, parents, n_entry, max_iters)
        rc = self._lib.memstore_retrieve_ann_users(self._h, _dev_ptr(queries, self.emb_torch_dtype, "queries"),
                                                   _dev_ptr(query_users, torch.int32, "query_users"), nq, k, C.byref(prm),
                                                   _dev_ptr(out_ids, torch.int32, "out_ids"), _dev_ptr(out_scores, torch.float32, "out_scores"),
                                                   _dev_ptr(counters, torch.int32, "counters"), _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return (out_ids, out_scores, counters) if want_counters else (out_ids, out_scores)

    def retrieve_static(self, queries, k, query_users=None, out_ids=None, out_scores=None, want_scores=True, stream=None):
        """``retrieve`` through the entry point that never allocates device memory, for callers that cannot let the
        library call cudaMalloc while serving (an engine that has claimed nearly all of HBM, a loop that cannot
        take the device-wide stall of an allocation).  Scratch is a fixed 4 MiB array inside the library shared by
        all such calls on the device, so the caller must not let two of them overlap on the GPU; sizes beyond
        1024 queries or 2^20 scores are refused.  Pass ``out_ids`` / ``out_scores`` to keep torch from allocating
        too."""
        nq = queries.shape[0]
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
        if out_scores is None and want_scores:
            out_scores = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
        rc = self._lib.memstore_retrieve_static(self._h, _dev_ptr(queries, self.emb_torch_dtype, "queries"),
                                                _dev_ptr(query_users, torch.int32, "query_users"), nq, k,
                                                _dev_ptr(out_ids, torch.int32, "out_ids"),
                                                _dev_ptr(out_scores, torch.float32, "out_scores"), _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out_ids, out_scores

    def inject(self, fact_ids, start_pos, block_tables, cache: PagedCache, out_n_tokens=None, out_status=None,
               out_slot_mapping=None, flags=0, stream=None):  # fmt: skip
        nreq, k = fact_ids.shape
        dev = fact_ids.device
        if out_n_tokens is None:
            out_n_tokens = torch.empty(nreq, dtype=torch.int32, device=dev)
        if out_status is None:
            out_status = torch.empty(nreq, dtype=torch.int32, device=dev)
        cs = cache._struct()
        rc = self._lib.memstore_inject(self._h, _dev_ptr(fact_ids, torch.int32, "fact_ids"), nreq, k,
                                       _dev_ptr(start_pos, torch.int32, "start_pos"),
                                       _dev_ptr(block_tables, torch.int32, "block_tables"), block_tables.shape[1],
                                       C.byref(cs), _dev_ptr(out_n_tokens, torch.int32, "out_n_tokens"),
                                       _dev_ptr(out_status, torch.int32, "out_status"),
                                       _dev_ptr(out_slot_mapping, torch.int64, "out_slot_mapping"),
                                       out_slot_mapping.shape[1] if out_slot_mapping is not None else 0,
                                       flags, _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out_n_tokens, out_status

    def retrieve_inject(self, queries, k, start_pos, block_tables, cache: PagedCache, query_users=None, out_ids=None,
                        out_scores=None, out_n_tokens=None, out_status=None, out_slot_mapping=None, flags=0, stream=None):  # fmt: skip
        """``retrieve`` then ``inject`` of every query's ids (query q = request q) in one call."""
        nq = queries.shape[0]
        dev = queries.device
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=dev)
        if out_n_tokens is None:
            out_n_tokens = torch.empty(nq, dtype=torch.int32, device=dev)
        if out_status is None:
            out_status = torch.empty(nq, dtype=torch.int32, device=dev)
        cs = cache._struct()
        rc = self._lib.memstore_retrieve_inject(
            self._h, _dev_ptr(queries, self.emb_torch_dtype, "queries"), _dev_ptr(query_users, torch.int32, "query_users"), nq,
            k, _dev_ptr(start_pos, torch.int32, "start_pos"), _dev_ptr(block_tables, torch.int32, "block_tables"),
            block_tables.shape[1], C.byref(cs), _dev_ptr(out_ids, torch.int32, "out_ids"),
            _dev_ptr(out_scores, torch.float32, "out_scores"), _dev_ptr(out_n_tokens, torch.int32, "out_n_tokens"),
            _dev_ptr(out_status, torch.int32, "out_status"), _dev_ptr(out_slot_mapping, torch.int64, "out_slot_mapping"),
            out_slot_mapping.shape[1] if out_slot_mapping is not None else 0, flags, _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out_ids, out_n_tokens, out_status

    def serve_host(self, query, k, start_pos, block_table, cache: PagedCache, out, user=0, flags=0, stream=None):
        """One request from HOST buffers (numpy arrays or CPU tensors): ``query`` [emb_dim], ``block_table`` int32
        [max_blocks]; ``out`` int32 [k + 2] receives ids, then the token count, then the status word."""
        import numpy as np

        def host_ptr(a, dtype):
            if isinstance(a, torch.Tensor):
                assert not a.is_cuda and a.is_contiguous() and a.dtype == dtype
                return C.c_void_p(a.data_ptr())
            assert isinstance(a, np.ndarray) and a.flags.c_contiguous
            return C.c_void_p(a.ctypes.data)

        cs = cache._struct()
        o = host_ptr(out, torch.int32)
        rc = self._lib.memstore_serve_host(self._h, host_ptr(query, self.emb_torch_dtype), user, k, int(start_pos),
                                           host_ptr(block_table, torch.int32), int(block_table.shape[-1]), C.byref(cs), flags,
                                           o, C.c_void_p(o.value + 4 * k), C.c_void_p(o.value + 4 * k + 4),
                                           _stream_ptr(stream))  # fmt: skip
        self._check(rc)
        return out

    def set_profile_events(self, before_copy=None, after_copy=None):
        """torch.cuda.Event pair (created with enable_timing=True and already recorded once so that they own a
        CUDA event) recorded around the copy kernel of every inject; (None, None) switches it off."""
        if before_copy is None and after_copy is None:
            self._check(self._lib.memstore_set_profile_events(self._h, None, None))
            self._prof = None
            return
        self._prof = (before_copy, after_copy)
        self._check(self._lib.memstore_set_profile_events(self._h, C.c_void_p(before_copy.cuda_event), C.c_void_p(after_copy.cuda_event)))

    def set_profile_repeats(self, n: int):
        """Measurement aid: launches of the copy kernel per inject call while profile events are set (see the header)."""
        self._check(self._lib.memstore_set_profile_repeats(self._h, int(n)))

    def stats(self) -> dict:
        st = _Stats()
        self._check(self._lib.memstore_stats(self._h, C.byref(st)))
        return {n: getattr(st, n) for n, _ in _Stats._fields_}

    def last_error(self) -> str:
        return self._lib.memstore_last_error(self._h).decode()
