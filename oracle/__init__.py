"""ctypes front end of the CPU oracle (``memoracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA library and its Python binding never
import this package, and this package imports nothing from them.

Every function marshals numpy arrays into the C routines and returns numpy
arrays; no arithmetic of the method happens in Python here.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_DIR = Path(__file__).resolve().parent
_SRC = _DIR / "memoracle.c"
_LIB = _DIR / "libmemoracle.so"

F32, F16 = 0, 1

OK = 0
ERR_ARG, ERR_BLOCK_TABLE, ERR_BLOCK_ID, ERR_FACT_ID, ERR_NOMEM = -1, -2, -3, -4, -5


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle returned {code}")
        self.code = code


def build(force: bool = False) -> Path:
    """Compile ``memoracle.c`` into ``libmemoracle.so`` next to it (gcc, -O3, OpenMP)."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-std=c11", "-O3", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra", str(_SRC), "-o", str(tmp), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_LIB))
        p, i32, i64, dbl = C.c_void_p, C.c_int, C.c_int64, C.c_double
        L.oracle_kv_bytes.restype = i64
        L.oracle_kv_bytes.argtypes = [i64] * 5
        L.oracle_max_threads.restype = i32
        L.oracle_scores.restype = i32
        L.oracle_scores.argtypes = [p, i32, i64, i32, p, p, i32]
        L.oracle_retrieve.restype = i32
        L.oracle_retrieve.argtypes = [p, i32, i64, i32, p, p, i32, i32, p, p, i32]
        L.oracle_inv_freq.restype = None
        L.oracle_inv_freq.argtypes = [i32, dbl, p]
        L.oracle_rope_rows.restype = i32
        L.oracle_rope_rows.argtypes = [p, i64, i32, p, dbl, i32, p, p]
        L.oracle_inject.restype = i32
        L.oracle_inject.argtypes = (
            [p, i32, i64, p, p, p, p, i64, i32, i32, i32, dbl, i32, p, i64, p, i64, i32, i64, i32, i32]
            + [p] * 7
            + [i64] * 4
            + [i32]
        )
        L.oracle_scores_f32.restype = i32
        L.oracle_scores_f32.argtypes = [p, i32, i64, i32, p, p]
        L.oracle_knn_graph.restype = i32
        L.oracle_knn_graph.argtypes = [p, i32, i64, i32, i32, p, i32]
        L.oracle_graph_append.restype = i32
        L.oracle_graph_append.argtypes = [p, i32, i64, i64, i32, p, i32, p, i32]
        L.oracle_ann_search.restype = i32
        L.oracle_ann_search.argtypes = [p, i32, i64, i32, p, i32, p, i32, i32, i32, i32, i32, p, p, p, p]
        L.oracle_ann_search_exact.restype = i32
        L.oracle_ann_search_exact.argtypes = L.oracle_ann_search.argtypes + [p]
        L.oracle_inject_ex.restype = i32
        L.oracle_inject_ex.argtypes = L.oracle_inject.argtypes + [i32, C.c_float, C.c_float, p, p]
        L.oracle_rope_rows_partial.restype = i32
        L.oracle_rope_rows_partial.argtypes = [p, i64, i32, i32, p, dbl, i32, p, p]
        L.oracle_inv_freq_llama3.restype = i32
        L.oracle_inv_freq_llama3.argtypes = [i32, dbl, dbl, dbl, dbl, dbl, p]
        for name in ("oracle_bf16_from_double", "oracle_bf16_to_double", "oracle_f16_to_double", "oracle_e4m3_from_double",
                     "oracle_e4m3_to_double"):  # fmt: skip
            getattr(L, name).restype = None
            getattr(L, name).argtypes = [p, i64, p]
        L.oracle_retrieve_masked.restype = i32
        L.oracle_retrieve_masked.argtypes = [p, i32, i64, i32, p, p, p, i32, i32, p, p, i32]
        L.oracle_knn_graph_masked.restype = i32
        L.oracle_knn_graph_masked.argtypes = [p, i32, i64, i32, i32, p, p, i32]
        L.oracle_ann_search_masked.restype = i32
        L.oracle_ann_search_masked.argtypes = [p, i32, i64, i32, p, i32, p, i32, i32, i32, i32, i32, i32, p, p, p, p, p, p]
        L.oracle_e4m3_from_scaled_bf16.restype = None
        L.oracle_e4m3_from_scaled_bf16.argtypes = [p, i64, C.c_float, p]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _emb_dtype(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float16:
        return F16
    raise TypeError(f"embeddings must be float32 or float16, got {a.dtype}")


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def kv_bytes(L: int, c: int, h: int, d: int, b: int) -> int:
    return int(lib().oracle_kv_bytes(L, c, h, d, b))


def bf16_from_double(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_bf16_from_double(_ptr(x), x.size, _ptr(out))
    return out


def bf16_to_double(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.uint16)
    out = np.empty(x.shape, dtype=np.float64)
    lib().oracle_bf16_to_double(_ptr(x), x.size, _ptr(out))
    return out


def f16_to_double(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x).view(np.uint16)
    out = np.empty(x.shape, dtype=np.float64)
    lib().oracle_f16_to_double(_ptr(x), x.size, _ptr(out))
    return out


def e4m3_from_double(x: np.ndarray) -> np.ndarray:
    """Round to the 8-bit e4m3 format (nearest even, one step, saturating at +-448)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint8)
    lib().oracle_e4m3_from_double(_ptr(x), x.size, _ptr(out))
    return out


def e4m3_from_scaled_bf16(bits: np.ndarray, scale: float) -> np.ndarray:
    """Codes of an 8-bit cache that holds value / scale: binary32(bf16 value) / scale in binary32, rounded once to e4m3."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.uint8)
    lib().oracle_e4m3_from_scaled_bf16(_ptr(bits), bits.size, float(scale), _ptr(out))
    return out


def e4m3_to_double(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.uint8)
    out = np.empty(x.shape, dtype=np.float64)
    lib().oracle_e4m3_to_double(_ptr(x), x.size, _ptr(out))
    return out


def scores(emb: np.ndarray, query: np.ndarray, n_threads: int = 0) -> np.ndarray:
    """Double-precision inner product of one query with every row of ``emb``."""
    emb = np.ascontiguousarray(emb)
    query = np.ascontiguousarray(query, dtype=emb.dtype).reshape(-1)
    n, e = emb.shape
    assert query.size == e
    out = np.empty(n, dtype=np.float64)
    if n:
        rc = lib().oracle_scores(_ptr(emb), _emb_dtype(emb), n, e, _ptr(query), _ptr(out), n_threads)
        if rc:
            raise OracleError(rc)
    return out


def _mask(removed, n):
    if removed is None:
        return None
    removed = np.ascontiguousarray(removed).astype(np.uint8)
    assert removed.size == n
    return removed


def retrieve(emb: np.ndarray, queries: np.ndarray, k: int, row_ids: np.ndarray | None = None, n_threads: int = 0, removed=None):
    """Top-k by (score descending, id ascending); returns (ids int32 [nq,k], scores float32 [nq,k]).
    ``removed``: boolean per row; removed rows are never returned."""
    emb = np.ascontiguousarray(emb)
    queries = np.ascontiguousarray(queries, dtype=emb.dtype)
    if queries.ndim == 1:
        queries = queries[None]
    n, e = emb.shape
    nq = queries.shape[0]
    if row_ids is not None:
        row_ids = np.ascontiguousarray(row_ids, dtype=np.int32)
        assert row_ids.size == n
    ids = np.empty((nq, k), dtype=np.int32)
    sc = np.empty((nq, k), dtype=np.float32)
    rc = lib().oracle_retrieve_masked(
        _ptr(emb), _emb_dtype(emb), n, e, _ptr(row_ids), _ptr(_mask(removed, n)), _ptr(queries), nq, k, _ptr(ids), _ptr(sc), n_threads
    )
    if rc:
        raise OracleError(rc)
    return ids, sc


def scores_f32(emb: np.ndarray, query: np.ndarray) -> np.ndarray:
    """Inner products in binary32 with the fixed lane order that the graph search compares scores in."""
    emb = np.ascontiguousarray(emb)
    query = np.ascontiguousarray(query, dtype=emb.dtype).reshape(-1)
    out = np.empty(emb.shape[0], dtype=np.float32)
    rc = lib().oracle_scores_f32(_ptr(emb), _emb_dtype(emb), emb.shape[0], emb.shape[1], _ptr(query), _ptr(out))
    if rc:
        raise OracleError(rc)
    return out


def knn_graph(emb: np.ndarray, deg: int, n_threads: int = 0, removed=None) -> np.ndarray:
    """Exact k-nearest-neighbour graph by inner product: int32 [n, deg], best first, -1 padded; ``removed`` rows are
    nobody's neighbours."""
    emb = np.ascontiguousarray(emb)
    out = np.empty((emb.shape[0], deg), dtype=np.int32)
    rc = lib().oracle_knn_graph_masked(_ptr(emb), _emb_dtype(emb), emb.shape[0], emb.shape[1], deg, _ptr(_mask(removed, emb.shape[0])),
                                       _ptr(out), n_threads)  # fmt: skip
    if rc:
        raise OracleError(rc)
    return out


def graph_append(emb: np.ndarray, old_graph: np.ndarray, n_threads: int = 0) -> np.ndarray:
    """The graph after rows ``old_graph.shape[0]`` .. ``emb.shape[0] - 1`` have been appended: exact lists for the new
    rows; an old row is offered the new rows that list it and keeps the best ``deg`` of old list + offers."""
    emb = np.ascontiguousarray(emb)
    old_graph = np.ascontiguousarray(old_graph, dtype=np.int32)
    n_old, deg = old_graph.shape
    out = np.empty((emb.shape[0], deg), dtype=np.int32)
    rc = lib().oracle_graph_append(_ptr(emb), _emb_dtype(emb), n_old, emb.shape[0], emb.shape[1], _ptr(old_graph), deg, _ptr(out), n_threads)
    if rc:
        raise OracleError(rc)
    return out


class AnnResult:
    def __init__(self, ids, scores, iters, scored, margin=None):
        self.ids, self.scores, self.iters, self.scored = ids, scores, iters, scored
        self.margin = margin  # exact search only: smallest score difference that decided a step, per query


def ann_search(emb: np.ndarray, graph: np.ndarray, queries: np.ndarray, k: int, beam: int = 64, parents: int = 8,
               n_entry: int = 64, max_iters: int = 32, exact: bool = False, removed=None) -> AnnResult:  # fmt: skip
    """Beam search over ``graph`` for each query: ids / scores [nq, k], steps taken and rows scored per query.
    ``exact``: rank by the double-precision inner products (and report the decision margin of every query) instead of
    the binary32 lane sums."""
    emb = np.ascontiguousarray(emb)
    graph = np.ascontiguousarray(graph, dtype=np.int32)
    queries = np.ascontiguousarray(queries, dtype=emb.dtype).reshape(-1, emb.shape[1])
    nq = queries.shape[0]
    ids = np.empty((nq, k), dtype=np.int32)
    sc = np.empty((nq, k), dtype=np.float32)
    iters = np.zeros(nq, dtype=np.int32)
    scored = np.zeros(nq, dtype=np.int64)
    margin = np.full(nq, np.inf) if exact else None
    removed = _mask(removed, emb.shape[0])
    for q in range(nq):
        it, ns = C.c_int32(0), C.c_int64(0)
        if removed is not None:
            mg = C.c_double(0.0)
            rc = lib().oracle_ann_search_masked(_ptr(emb), _emb_dtype(emb), emb.shape[0], emb.shape[1], _ptr(graph), graph.shape[1],
                                                _ptr(queries[q]), k, beam, parents, n_entry, max_iters, int(exact), _ptr(removed),
                                                _ptr(ids[q]), _ptr(sc[q]), C.byref(it), C.byref(ns), C.byref(mg))  # fmt: skip
            if rc:
                raise OracleError(rc)
            iters[q], scored[q] = it.value, ns.value
            if exact:
                margin[q] = mg.value
            continue
        if exact:
            mg = C.c_double(0.0)
            rc = lib().oracle_ann_search_exact(_ptr(emb), _emb_dtype(emb), emb.shape[0], emb.shape[1], _ptr(graph), graph.shape[1],
                                               _ptr(queries[q]), k, beam, parents, n_entry, max_iters, _ptr(ids[q]), _ptr(sc[q]),
                                               C.byref(it), C.byref(ns), C.byref(mg))  # fmt: skip
            if rc:
                raise OracleError(rc)
            iters[q], scored[q], margin[q] = it.value, ns.value, mg.value
            continue
        rc = lib().oracle_ann_search(_ptr(emb), _emb_dtype(emb), emb.shape[0], emb.shape[1], _ptr(graph), graph.shape[1],
                                     _ptr(queries[q]), k, beam, parents, n_entry, max_iters, _ptr(ids[q]), _ptr(sc[q]),
                                     C.byref(it), C.byref(ns))  # fmt: skip
        if rc:
            raise OracleError(rc)
        iters[q], scored[q] = it.value, ns.value
    return AnnResult(ids, sc, iters, scored, margin)


def inv_freq(D: int, theta: float) -> np.ndarray:
    out = np.empty(D // 2, dtype=np.float32)
    lib().oracle_inv_freq(D, float(theta), _ptr(out))
    return out


def inv_freq_llama3(R: int, theta: float, factor=8.0, low_freq_factor=1.0, high_freq_factor=4.0, original_max=8192.0) -> np.ndarray:
    """The rescaled frequency table of the Llama-3.1 family for a rotary dimension ``R``."""
    out = np.empty(R // 2, dtype=np.float32)
    rc = lib().oracle_inv_freq_llama3(R, float(theta), float(factor), float(low_freq_factor), float(high_freq_factor),
                                      float(original_max), _ptr(out))  # fmt: skip
    if rc:
        raise OracleError(rc)
    return out


def rope_rows(x: np.ndarray, pos: np.ndarray, theta: float, style: int = 0, inv_freq_override=None, rotary_dim: int = 0) -> np.ndarray:
    """Rotate rows of ``x`` ([n, D] float64), row r at position ``pos[r]``; ``rotary_dim``: only the first
    so many coordinates rotate (0 = all)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    n, D = x.shape
    pos = np.ascontiguousarray(np.broadcast_to(np.asarray(pos, dtype=np.int64), (n,)))
    if inv_freq_override is not None:
        inv_freq_override = np.ascontiguousarray(inv_freq_override, dtype=np.float32)
        assert inv_freq_override.size == (rotary_dim or D) // 2
    y = np.empty_like(x)
    if rotary_dim:
        rc = lib().oracle_rope_rows_partial(_ptr(x), n, D, rotary_dim, _ptr(pos), float(theta), style, _ptr(inv_freq_override), _ptr(y))
    else:
        rc = lib().oracle_rope_rows(_ptr(x), n, D, _ptr(pos), float(theta), style, _ptr(inv_freq_override), _ptr(y))
    if rc:
        raise OracleError(rc)
    return y


def slots(ids, fact_len, start_pos, block_table, bs, num_blocks):
    """Positions and slots only (no K/V touched): returns (m, slots[m]) for facts ``ids`` in placement order."""
    ids = np.ascontiguousarray(ids, dtype=np.int32).reshape(-1)
    fact_len = np.ascontiguousarray(fact_len, dtype=np.int32)
    fact_offset = np.zeros(fact_len.size, dtype=np.int64)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32).reshape(-1)
    valid = ids[(ids >= 0) & (ids < fact_len.size)]
    out = np.empty(int(fact_len[valid].sum()), dtype=np.int64)
    dummy = np.zeros(1, dtype=np.uint16)
    m = C.c_int64(0)
    rc = lib().oracle_inject(
        _ptr(ids), ids.size, fact_len.size, _ptr(fact_offset), _ptr(fact_len), _ptr(dummy), _ptr(dummy), 1 << 62,
        1, 1, 2, 1.0, 0, None, int(start_pos), _ptr(block_table), block_table.size, bs, num_blocks, 0, 0,
        C.byref(m), _ptr(out), None, None, None, None, None, 0, 0, 0, 0, 1,
    )  # fmt: skip
    if rc:
        raise OracleError(rc)
    return m.value, out


class InjectResult:
    """m, slots [m], k_ref float64 / k_bf16 uint16 / v uint16, each [nl, m, H, D]."""

    def __init__(self, m, slots, k_ref, k_bf16, v, k_fp8=None, v_fp8=None):
        self.m, self.slots, self.k_ref, self.k_bf16, self.v = m, slots, k_ref, k_bf16, v
        self.k_fp8, self.v_fp8 = k_fp8, v_fp8  # uint8 e4m3 codes of K / k_scale and V / v_scale, when scales were given


def inject(
    ids,
    fact_offset,
    fact_len,
    k_pre,
    v,
    theta,
    start_pos,
    block_table,
    bs,
    num_blocks,
    style=0,
    inv_freq_override=None,
    layers=None,
    want_ref=True,
    k_cache=None,
    v_cache=None,
    cache_strides=None,
    n_threads=0,
    rotary_dim=0,
    k_scale=None,
    v_scale=None,
) -> InjectResult:
    """Compose facts ``ids`` (placement order) at ``start_pos`` and place them through ``block_table``.

    ``k_pre`` / ``v``: uint16 (bf16 bits) arrays [n_layers, store_tokens, H, D] on the host.
    ``k_cache`` / ``v_cache``: optional uint16 host images of the paged cache, written in place using
    ``cache_strides = (layer, block, token, head)`` in elements.
    ``rotary_dim``: only the first so many coordinates of a head rotate (0 = all).  ``k_scale`` / ``v_scale``:
    also return the e4m3 codes of an 8-bit cache that holds K / k_scale and V / v_scale.
    """
    ids = np.ascontiguousarray(ids, dtype=np.int32).reshape(-1)
    fact_offset = np.ascontiguousarray(fact_offset, dtype=np.int64)
    fact_len = np.ascontiguousarray(fact_len, dtype=np.int32)
    assert k_pre.dtype == np.uint16 and v.dtype == np.uint16 and k_pre.shape == v.shape
    k_pre = np.ascontiguousarray(k_pre)
    v = np.ascontiguousarray(v)
    n_layers, store_tokens, H, D = k_pre.shape
    block_table = np.ascontiguousarray(block_table, dtype=np.int32).reshape(-1)
    l0, l1 = (0, n_layers) if layers is None else layers
    nl = l1 - l0
    if inv_freq_override is not None:
        inv_freq_override = np.ascontiguousarray(inv_freq_override, dtype=np.float32)
    valid = ids[(ids >= 0) & (ids < fact_len.size)]
    m_guess = int(fact_len[valid].sum())
    slots = np.empty(m_guess, dtype=np.int64)
    shape = (nl, m_guess, H, D)
    k_ref = np.empty(shape, dtype=np.float64) if want_ref else None
    k_bf16 = np.empty(shape, dtype=np.uint16)
    v_out = np.empty(shape, dtype=np.uint16)
    m = C.c_int64(0)
    strides = (0, 0, 0, 0)
    if k_cache is not None or v_cache is not None:
        assert cache_strides is not None
        strides = tuple(int(s) for s in cache_strides)
        for c_ in (k_cache, v_cache):
            assert c_ is None or (c_.dtype == np.uint16 and c_.flags.c_contiguous)
    k_fp8 = np.empty(shape, dtype=np.uint8) if k_scale is not None else None
    v_fp8 = np.empty(shape, dtype=np.uint8) if v_scale is not None else None
    rc = lib().oracle_inject_ex(
        _ptr(ids), ids.size, fact_len.size, _ptr(fact_offset), _ptr(fact_len), _ptr(k_pre), _ptr(v), store_tokens,
        n_layers, H, D, float(theta), style, _ptr(inv_freq_override), int(start_pos), _ptr(block_table),
        block_table.size, bs, num_blocks, l0, l1, C.byref(m), _ptr(slots), _ptr(k_ref), _ptr(k_bf16), _ptr(v_out),
        _ptr(k_cache), _ptr(v_cache), *strides, n_threads, int(rotary_dim), float(k_scale or 0.0), float(v_scale or 0.0),
        _ptr(k_fp8), _ptr(v_fp8),
    )  # fmt: skip
    if rc:
        raise OracleError(rc)
    assert m.value == m_guess
    return InjectResult(m.value, slots, k_ref, k_bf16, v_out, k_fp8, v_fp8)
