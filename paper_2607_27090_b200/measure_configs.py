"""Timing of the batched workload configurations (many queries / many requests per call) on one GPU.

    python -m paper_2607_27090_b200.measure_configs --config users100|stress1m|gqa14b|llama8b [--iters 20]

``bench.py`` times the headline configuration (one request at k = 50).  This module times the others the same
way (CUDA events on one stream, warm-up first, inputs already in HBM) and prints one JSON line per
configuration: microseconds of the batched retrieve call and of the batched inject call, bytes scanned / moved,
and the rates they imply.  No step of the method runs here; the hot set of a configuration with partial
residency (a store-construction input) comes from the library's own retrieval on an embedding-only store.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import memstore as M
from . import synth, workload


def free_gib(device) -> float:
    free, _ = torch.cuda.mem_get_info(device)
    return free / 2**30


def candidate_hot_ids(emb: np.ndarray, queries: np.ndarray, per_query: int, users: np.ndarray | None = None, per_user: int = 0,
                      device="cuda"):  # fmt: skip
    """Ids that a request may name (a store-construction input: facts outside this set get no K/V): per query the
    ``per_query`` best facts of its user's segment, taken from the LIBRARY's own exact retrieval on a temporary
    embedding-only store, so that no scoring or selection is restated here.  A superset of every top-k list with
    k <= per_query."""
    dev = torch.device(device)
    n_users = 1 if users is None else int(per_user and emb.shape[0] // per_user)
    seg = emb.shape[0] // n_users
    tdt = torch.float32 if emb.dtype == np.float32 else torch.float16
    store = M.MemStore(device=dev.index or 0, n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=emb.shape[1], emb_dtype=tdt,
                       rope_theta=1e4, n_users=n_users, max_facts_per_user=seg, max_kv_tokens=0)  # fmt: skip
    for u in range(n_users):
        for a in range(u * seg, (u + 1) * seg, 65536):
            b = min((u + 1) * seg, a + 65536)
            store.add_facts(torch.from_numpy(emb[a:b]).to(dev), [0] * (b - a), user=u)
    q_dev = torch.from_numpy(queries).to(dev)
    u_dev = torch.from_numpy(np.asarray(users, np.int32)).to(dev) if users is not None else None
    ids, _ = store.retrieve(q_dev, per_query, query_users=u_dev)
    torch.cuda.synchronize(dev)
    hot = sorted({int(i) for i in ids.cpu().numpy().reshape(-1) if i >= 0})
    store.close()
    return hot


def measure_retrieve_only(name: str, iters: int, seed: int = 0):
    """Batched retrieval alone on an embedding-only store (no K/V, no cache): a few GB at most, for profiler captures."""
    s = synth.CONFIGS[name]
    dev = torch.device("cuda")
    total = s.n_facts * s.n_users
    emb = synth.embeddings(seed, total, s.emb_dim, s.emb_dtype)
    queries = synth.queries(seed, s.nq, s.emb_dim, s.emb_dtype)
    tdt = torch.float32 if s.emb_dtype == "float32" else torch.float16
    store = M.MemStore(n_layers=s.n_layers, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, emb_dim=s.emb_dim, emb_dtype=tdt,
                       rope_theta=s.rope_theta, n_users=s.n_users, max_facts_per_user=s.n_facts, max_kv_tokens=0)  # fmt: skip
    for u in range(s.n_users):
        for a in range(u * s.n_facts, (u + 1) * s.n_facts, 65536):
            b = min((u + 1) * s.n_facts, a + 65536)
            store.add_facts(torch.from_numpy(emb[a:b]).to(dev), [0] * (b - a), user=u)
    q_dev = torch.from_numpy(queries).to(dev)
    u_dev = torch.arange(s.n_users, dtype=torch.int32, device=dev) if s.n_users > 1 else None
    ids = torch.empty((s.nq, s.k), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(2):
        store.retrieve(q_dev, s.k, query_users=u_dev, out_ids=ids, want_scores=False, stream=stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(iters):
        store.retrieve(q_dev, s.k, query_users=u_dev, out_ids=ids, want_scores=False, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / iters
    line = {"config": name, "mode": "retrieve only", "queries_per_call": s.nq, "k": s.k, "facts_scanned": total,
            "retrieve_us": us, "retrieve_emb_gbs": workload.emb_bytes_scanned(s, total) / (us * 1e-6) / 1e9,
            "kernel_timeouts": store.stats()["kernel_timeouts"]}  # fmt: skip
    st = store.stats()
    if st["filter_list_queries"] + st["filter_list_fallbacks"]:
        line["filter_list"] = {"queries": st["filter_list_queries"], "fallbacks": st["filter_list_fallbacks"],
                               "rows_per_query": st["filter_list_rows"] / max(1, st["filter_list_queries"])}  # fmt: skip
    store.close()
    return line


def measure_host_tier(iters: int, seed: int = 0, n_facts: int = 400, ks=(5, 10, 20, 50)):
    """The Llama-3.1-8B KV shape with every fact's K/V in the pinned host arena (the CPU-offloaded store): injection
    of k facts read over PCIe by the copy kernel.  A shrunken store (n_facts) keeps the pinned allocation near 2 GB."""
    s = synth.CONFIGS["llama8b"]
    dev = torch.device("cuda")
    lens = synth.fact_lengths(seed, n_facts, s.len_lo, s.len_hi)
    emb = synth.embeddings(seed, n_facts, s.emb_dim, s.emb_dtype)
    T = int(lens.sum())
    store = M.MemStore(n_layers=s.n_layers, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, emb_dim=s.emb_dim,
                       rope_theta=s.rope_theta, max_facts_per_user=n_facts, max_kv_tokens=0, max_host_kv_tokens=T)  # fmt: skip
    g = torch.Generator().manual_seed(seed)
    for a in range(0, n_facts, 50):
        b = min(n_facts, a + 50)
        t = int(lens[a:b].sum())
        kv = torch.randn((2, s.n_layers, t, s.n_kv_heads, s.head_dim), generator=g, dtype=torch.float32).to(torch.bfloat16)
        store.add_facts_host(torch.from_numpy(emb[a:b]).to(dev), lens[a:b], kv[0].contiguous(), kv[1].contiguous())
    lines = []
    rng = np.random.default_rng(seed)
    for k in ks:
        per_req = workload.blocks_per_request(s, k)
        cache = M.PagedCache.allocate(s.n_layers, max(1024, per_req * 4), s.block_size, s.n_kv_heads, s.head_dim, dev)
        tables = torch.from_numpy(synth.block_tables(seed, cache.num_blocks, per_req, 4)).to(dev)
        ids = torch.from_numpy(np.stack([rng.choice(n_facts, k, replace=False) for _ in range(4)]).astype(np.int32)).to(dev)
        start = torch.full((1,), s.start_pos, dtype=torch.int32, device=dev)
        n_tok = torch.zeros(1, dtype=torch.int32, device=dev)
        stream = torch.cuda.current_stream()
        for i in range(3):
            store.inject(ids[i % 4 : i % 4 + 1], start, tables[i % 4 : i % 4 + 1], cache, out_n_tokens=n_tok, stream=stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m_sum = 0
        e0.record(stream)
        for i in range(iters):
            store.inject(ids[i % 4 : i % 4 + 1], start, tables[i % 4 : i % 4 + 1], cache, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        for i in range(4):
            m_sum += int(lens[ids[i].cpu().numpy()].sum())
        us = e0.elapsed_time(e1) * 1e3 / iters
        m = m_sum / 4
        lines.append({"config": "llama8b host tier", "k": k, "tokens": m, "inject_us": us,
                      "pcie_read_gbs": m * s.token_bytes / (us * 1e-6) / 1e9})  # fmt: skip
        del cache
    store.close()
    return lines


def measure_compose_cache(iters: int, seed: int = 0, n_facts: int = 400, ks=(5, 10, 20, 50)):
    """Host-tier store of the Llama-3.1-8B KV shape: a request composed from pinned host memory (miss: rows cross PCIe)
    against the same request repeated with the composition cache on (hit: an HBM-rate copy of the cached segment)."""
    s = synth.CONFIGS["llama8b"]
    dev = torch.device("cuda")
    lens = synth.fact_lengths(seed, n_facts, s.len_lo, s.len_hi)
    emb = synth.embeddings(seed, n_facts, s.emb_dim, s.emb_dtype)
    T = int(lens.sum())
    store = M.MemStore(n_layers=s.n_layers, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, emb_dim=s.emb_dim,
                       rope_theta=s.rope_theta, max_facts_per_user=n_facts, max_kv_tokens=0, max_host_kv_tokens=T)  # fmt: skip
    g = torch.Generator().manual_seed(seed)
    for a in range(0, n_facts, 50):
        b = min(n_facts, a + 50)
        t = int(lens[a:b].sum())
        kv = torch.randn((2, s.n_layers, t, s.n_kv_heads, s.head_dim), generator=g, dtype=torch.float32).to(torch.bfloat16)
        store.add_facts_host(torch.from_numpy(emb[a:b]).to(dev), lens[a:b], kv[0].contiguous(), kv[1].contiguous())
    lines = []
    rng = np.random.default_rng(seed)
    stream = torch.cuda.current_stream()
    for k in ks:
        per_req = workload.blocks_per_request(s, k)
        cache = M.PagedCache.allocate(s.n_layers, max(1024, per_req * 4), s.block_size, s.n_kv_heads, s.head_dim, dev)
        tables = torch.from_numpy(synth.block_tables(seed, cache.num_blocks, per_req, 4)).to(dev)
        ids = torch.from_numpy(rng.choice(n_facts, k, replace=False).astype(np.int32)[None]).to(dev)
        m = int(lens[ids.cpu().numpy()[0]].sum())
        start = torch.full((1,), s.start_pos, dtype=torch.int32, device=dev)

        def timed(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for i in range(n):
                store.inject(ids, start, tables[i % 4 : i % 4 + 1], cache, flags=M.INJECT_REVERSE, stream=stream)
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / n

        store.compose_cache(0)
        timed(2)
        miss_us = timed(max(2, iters // 4))
        store.compose_cache(2 * k * s.len_hi * s.token_bytes, k * s.len_hi)
        fill_us = timed(1)  # the first repetition records the segment
        hit_us = timed(iters)
        st = store.stats()
        lines.append({"config": "llama8b host tier, repeated request", "k": k, "tokens": m, "miss_us": miss_us, "recording_miss_us": fill_us,
                      "hit_us": hit_us, "hit_gbs": 2.0 * m * s.token_bytes / (hit_us * 1e-6) / 1e9, "hits": st["compose_cache_hits"],
                      "fills": st["compose_cache_fills"]})  # fmt: skip
        del cache
    store.close()
    return lines


def measure_permuted_chunks(iters: int, seed: int = 0, sizes=(1024, 2048, 4096, 8192, 16384, 32768), chunk: int = 64):
    """The shape of the paper's chunk-order experiment (appendix "Position independence and rotation fidelity") on the
    Llama-3.1-8B KV shape: fixed 64-token chunks injected
    in a fresh random order every time, 1K to 32K tokens per request (512 chunks = 4.3 GB of stored K/V)."""
    s = synth.CONFIGS["llama8b"]
    dev = torch.device("cuda")
    n_chunks = max(sizes) // chunk
    T = n_chunks * chunk
    store = M.MemStore(n_layers=s.n_layers, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, emb_dim=s.emb_dim, rope_theta=s.rope_theta,
                       max_facts_per_user=n_chunks, max_kv_tokens=T)  # fmt: skip
    emb = synth.embeddings(seed, n_chunks, s.emb_dim, s.emb_dtype)
    g = torch.Generator(device=dev).manual_seed(seed)
    for a in range(0, n_chunks, 32):
        b = min(n_chunks, a + 32)
        kv = torch.randn((2, s.n_layers, (b - a) * chunk, s.n_kv_heads, s.head_dim), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
        store.add_facts(torch.from_numpy(emb[a:b]).to(dev), [chunk] * (b - a), kv[0].contiguous(), kv[1].contiguous())
    bs = s.block_size
    nb = max(sizes) // bs + 8
    cache = M.PagedCache.allocate(s.n_layers, nb, bs, s.n_kv_heads, s.head_dim, dev)
    rng = np.random.default_rng(seed)
    table = torch.from_numpy(synth.block_tables(seed, nb, nb - 1, 1)).to(dev)
    start = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    lines = []
    for m in sizes:
        k = m // chunk
        orders = torch.from_numpy(np.stack([rng.permutation(n_chunks)[:k] for _ in range(4)]).astype(np.int32)).to(dev)
        for i in range(2):
            store.inject(orders[i : i + 1], start, table, cache, stream=stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(iters):
            store.inject(orders[i % 4 : i % 4 + 1], start, table, cache, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / iters
        lines.append({"config": "llama8b permuted 64-token chunks", "tokens": m, "chunks": k, "inject_us": us,
                      "inject_gbs": 2.0 * m * s.token_bytes / (us * 1e-6) / 1e9})  # fmt: skip
    store.close()
    return lines


def measure_variants(iters: int, seed: int = 0, n_facts: int = 400, k: int = 50):
    """Injection of k facts on the Llama-3.1-8B KV shape (a shrunken store: the traffic of a request does not depend on
    the store size) in the parameterisation variants: bf16 cache (the headline path), 8-bit e4m3 cache (half the
    write traffic), and rotation of the first 64 coordinates only."""
    s = synth.CONFIGS["llama8b"]
    dev = torch.device("cuda")
    lens = synth.fact_lengths(seed, n_facts, s.len_lo, s.len_hi)
    T = int(lens.sum())
    emb = synth.embeddings(seed, n_facts, s.emb_dim, s.emb_dtype)
    rng = np.random.default_rng(seed)
    per_req = workload.blocks_per_request(s, k)
    ids = torch.from_numpy(np.stack([rng.choice(n_facts, k, replace=False) for _ in range(4)]).astype(np.int32)).to(dev)
    m = float(np.mean([lens[ids[i].cpu().numpy()].sum() for i in range(4)]))
    lines = []
    for variant, rotary_dim, fp8 in (("bf16 cache", 0, False), ("e4m3 cache", 0, True), ("rotary_dim 64, bf16 cache", 64, False)):
        store = M.MemStore(n_layers=s.n_layers, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, emb_dim=s.emb_dim, rope_theta=s.rope_theta,
                           max_facts_per_user=n_facts, max_kv_tokens=T, rotary_dim=rotary_dim)  # fmt: skip
        g = torch.Generator(device=dev).manual_seed(seed)
        for a in range(0, n_facts, 50):
            b = min(n_facts, a + 50)
            t = int(lens[a:b].sum())
            kv = torch.randn((2, s.n_layers, t, s.n_kv_heads, s.head_dim), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
            store.add_facts(torch.from_numpy(emb[a:b]).to(dev), lens[a:b], kv[0].contiguous(), kv[1].contiguous())
        cache = M.PagedCache.allocate(s.n_layers, max(1024, per_req * 4), s.block_size, s.n_kv_heads, s.head_dim, dev, fp8=fp8,
                                      k_scale=0.05, v_scale=0.05)  # fmt: skip
        tables = torch.from_numpy(synth.block_tables(seed, cache.num_blocks, per_req, 4)).to(dev)
        start = torch.full((1,), s.start_pos, dtype=torch.int32, device=dev)
        stream = torch.cuda.current_stream()
        for i in range(3):
            store.inject(ids[i % 4 : i % 4 + 1], start, tables[i % 4 : i % 4 + 1], cache, stream=stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(iters):
            store.inject(ids[i % 4 : i % 4 + 1], start, tables[i % 4 : i % 4 + 1], cache, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / iters
        moved = m * s.token_bytes * (1.5 if fp8 else 2.0)  # read K and V (bf16), write both (one or two bytes per element)
        lines.append({"config": "llama8b " + variant, "k": k, "tokens": m, "inject_us": us, "bytes_moved": moved,
                      "inject_gbs": moved / (us * 1e-6) / 1e9})  # fmt: skip
        store.close()
        del cache
    return lines


def measure_ann(n: int, iters: int, seed: int = 0, dim: int = 1024, degree: int = 64, k: int = 50, intrinsic_dim: int = 32):
    """Graph index on an embedding-only store of ``n`` structured rows (low intrinsic dimension, queries near stored
    rows): build time, search time for 1 and for 64 queries, rows scored, recall against the exact retrieval of the
    same store, and the exact retrieval times beside them."""
    import time

    dev = torch.device("cuda")
    emb = synth.embeddings_low_rank(seed, n, dim, "float16", intrinsic_dim=intrinsic_dim)
    q = synth.queries_near_rows(seed, emb, 64)
    store = M.MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=dim, rope_theta=1e4, max_facts_per_user=n, max_kv_tokens=0)
    n_late = min(640, n // 10)  # these rows arrive after the build and are linked by graph_append
    for a in range(0, n - n_late, 65536):
        b = min(n - n_late, a + 65536)
        store.add_facts(torch.from_numpy(emb[a:b]).to(dev), [0] * (b - a))
    q_dev = torch.from_numpy(q).to(dev)
    stream = torch.cuda.current_stream()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    store.build_graph(degree, stream=stream)
    torch.cuda.synchronize()
    build_s = time.perf_counter() - t0
    store.add_facts(torch.from_numpy(emb[n - n_late :]).to(dev), [0] * n_late)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    store.graph_append(stream=stream)
    torch.cuda.synchronize()
    append_s = time.perf_counter() - t0

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(iters):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / iters

    ids_e = torch.empty((64, k), dtype=torch.int32, device=dev)
    ids_a = torch.empty((64, k), dtype=torch.int32, device=dev)
    exact_64 = timed(lambda: store.retrieve(q_dev, k, out_ids=ids_e, want_scores=False, stream=stream))
    exact_1 = timed(lambda: store.retrieve(q_dev[:1], k, out_ids=ids_e[:1], want_scores=False, stream=stream))
    store.retrieve(q_dev, k, out_ids=ids_e, want_scores=False, stream=stream)
    lines = []
    for beam in (64, 128, 256):
        L = max(beam, k)
        ann_64 = timed(lambda: store.retrieve_ann(q_dev, k, beam=L, out_ids=ids_a, want_scores=False, stream=stream))
        ann_1 = timed(lambda: store.retrieve_ann(q_dev[:1], k, beam=L, out_ids=ids_a[:1], want_scores=False, stream=stream))
        _, _, cnt = store.retrieve_ann(q_dev, k, beam=L, out_ids=ids_a, want_scores=False, want_counters=True, stream=stream)
        torch.cuda.synchronize()
        a, b = ids_a.cpu().numpy(), ids_e.cpu().numpy()
        recall = float(np.mean([len(set(a[i]) & set(b[i])) / k for i in range(64)]))
        lines.append({"config": f"graph index, {n} rows x {dim} fp16, degree {degree}", "k": k, "beam": L, "build_s": build_s,
                      "append_rows": n_late, "append_ms": append_s * 1e3,
                      "recall_at_k": recall, "ann_us_1_query": ann_1, "ann_us_64_queries": ann_64,
                      "exact_us_1_query": exact_1, "exact_us_64_queries": exact_64,
                      "mean_steps": float(cnt[:, 0].float().mean()), "mean_rows_scored": float(cnt[:, 1].float().mean())})  # fmt: skip
    store.close()
    return lines


def measure(name: str, iters: int, seed: int = 0, hot_per_user: int | None = None, pool_blocks: int | None = None,
            want_pool_blocks: int | None = None, headroom_gib: float = 6.0):  # fmt: skip
    """One batched configuration: the store is built as the configuration states it when the free device memory allows
    (hot subset of ``resident_per_user`` facts, ``want_pool_blocks`` cache blocks), else the hot subset and then the
    pool are halved until they fit; the sizes used are in the line."""
    s = synth.CONFIGS[name]
    dev = torch.device("cuda")
    total = s.n_facts * s.n_users
    emb = synth.embeddings(seed, total, s.emb_dim, s.emb_dtype)
    nq = s.nq
    queries = synth.queries(seed, nq, s.emb_dim, s.emb_dtype)
    k_inj = 50 if name == "stress1m" else s.k
    users = np.arange(s.n_users, dtype=np.int32) if s.n_users > 1 else None
    per_req = workload.blocks_per_request(s, k_inj)
    nb_min = max(1024, 1 << int(np.ceil(np.log2(per_req * nq))))  # every request of a call has its own blocks
    nb = pool_blocks or max(nb_min, want_pool_blocks or 0)
    mean_len = (s.len_lo + s.len_hi) / 2
    hot, note = None, "as configured"
    if s.resident_per_user is not None:
        hot = candidate_hot_ids(emb, queries, k_inj + 14, users, s.n_facts, dev)
        need_per_user = (len(hot) + s.n_users - 1) // s.n_users
        if hot_per_user is None:
            hot_per_user = max(s.resident_per_user, need_per_user)
        # what fits: store (hot facts) + pool + the embeddings, with some headroom for scratch
        emb_gib = workload.emb_bytes_scanned(s, total) / 2**30
        avail = free_gib(dev) - headroom_gib - emb_gib
        store_gib = lambda h: h * s.n_users * mean_len * 1.03 * s.token_bytes / 2**30  # noqa: E731
        pool_gib = lambda n: n * s.block_size * s.token_bytes / 2**30  # noqa: E731
        while pool_blocks is None and nb > nb_min and store_gib(hot_per_user) + pool_gib(nb) > avail:
            nb //= 2
            note = "pool halved to fit the free device memory"
        while hot_per_user > need_per_user and store_gib(hot_per_user) + pool_gib(nb) > avail:
            hot_per_user = max(need_per_user, hot_per_user // 2)
            note = "hot subset (and pool) reduced to fit the free device memory"
    wl = workload.build(name, seed=seed, device=dev, n_query_pool=nq, num_blocks=nb, resident_ids=hot, hot_per_user=hot_per_user,
                        emb=emb, queries=queries)  # fmt: skip
    store, cache = wl.store, wl.cache
    q_dev = torch.from_numpy(queries).to(dev)
    u_dev = torch.from_numpy(users).to(dev) if users is not None else None
    n_sets = 2
    tables = [torch.from_numpy(synth.block_tables(seed + t, cache.num_blocks, per_req, nq)).to(dev) for t in range(n_sets)]
    starts = torch.full((nq,), s.start_pos, dtype=torch.int32, device=dev)
    ids = torch.empty((nq, s.k), dtype=torch.int32, device=dev)
    n_tok = torch.zeros(nq, dtype=torch.int32, device=dev)
    status = torch.zeros(nq, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def retrieve():
        store.retrieve(q_dev, s.k, query_users=u_dev, out_ids=ids, want_scores=False, stream=stream)

    def inject(i):
        top = ids if k_inj == s.k else ids[:, :k_inj].contiguous()
        store.inject(top, starts, tables[i % n_sets], cache, out_n_tokens=n_tok, out_status=status, flags=M.INJECT_REVERSE, stream=stream)

    for i in range(3):
        retrieve()
        inject(i)
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0, "a request named a fact without K/V: the hot set was chosen too small"
    m_total = int(n_tok.sum())
    # retrieve and inject alternate on the stream without a host synchronise in between (the GPU stays busy, as in a
    # serving loop: an event pair around a call issued to an idle GPU would also time the host's launch path)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(iters)]
    for i in range(iters):
        evs[i][0].record(stream)
        retrieve()
        evs[i][1].record(stream)
        inject(i)
        evs[i][2].record(stream)
    torch.cuda.synchronize()
    t_r = [e[0].elapsed_time(e[1]) * 1e3 for e in evs]
    t_i = [e[1].elapsed_time(e[2]) * 1e3 for e in evs]
    ev = evs[0]
    # the retrieval call alone, back to back (no injection between two calls): a few calls first, so that the timed ones
    # start in the steady state, and enough of them that the first one's lone start does not weigh
    n_b2b = max(iters, 100)
    for i in range(5):
        retrieve()
    ev[0].record(stream)
    for i in range(n_b2b):
        retrieve()
    ev[1].record(stream)
    torch.cuda.synchronize()
    r_b2b = ev[0].elapsed_time(ev[1]) * 1e3 / n_b2b
    # the one call that does both (memstore_retrieve_inject), calls back to back, where the injection takes all k ids
    fused_us = None
    if k_inj == s.k:
        def fused(i):
            store.retrieve_inject(q_dev, s.k, starts, tables[i % n_sets], cache, query_users=u_dev, out_ids=ids, out_n_tokens=n_tok,
                                  out_status=status, flags=M.INJECT_REVERSE, stream=stream)  # fmt: skip

        for i in range(2):
            fused(i)
        ev[0].record(stream)
        for i in range(iters):
            fused(i)
        ev[1].record(stream)
        torch.cuda.synchronize()
        fused_us = ev[0].elapsed_time(ev[1]) * 1e3 / iters
    r_us, i_us = float(np.median(t_r)), float(np.median(t_i))
    emb_bytes = workload.emb_bytes_scanned(s, total)
    kv_bytes = workload.kv_bytes_moved(s, m_total)
    flops = 2.0 * total * s.emb_dim * nq if s.n_users == 1 else 2.0 * total * s.emb_dim
    line = {
        "config": name, "queries_per_call": nq, "k": s.k, "k_injected": k_inj, "requests_per_call": nq,
        "facts_scanned": total, "tokens_injected": m_total, "pool_blocks": cache.num_blocks,
        "resident_facts": int((wl.lens > 0).sum()), "sizes_note": note,
        "store_gib": float(wl.lens.sum()) * s.token_bytes / 2**30, "pool_gib": cache.num_blocks * s.block_size * s.token_bytes / 2**30,
        "retrieve_us": r_us, "retrieve_back_to_back_us": r_b2b, "retrieve_inject_call_us": fused_us, "retrieve_emb_gbs": emb_bytes / (r_us * 1e-6) / 1e9,
        "retrieve_tflops": flops / (r_us * 1e-6) / 1e12,
        "inject_us": i_us, "inject_gbs": kv_bytes / (i_us * 1e-6) / 1e9,
        "us_per_request": (r_us + i_us) / nq,
        "kernel_timeouts": store.stats()["kernel_timeouts"],
    }  # fmt: skip
    store.close()
    del wl, cache, tables
    torch.cuda.empty_cache()
    return line


# the pool sizes the configurations state (blocks); others derive theirs from the requests
CONFIGURED_POOL_BLOCKS = {"users100": 65536, "stress1m": 16384}


def measure_all(peak_gbs: float, budget_s: float = 90.0, iters: int = 10, seed: int = 0, names=("gqa14b", "users100", "stress1m")):
    """The batched configurations one after the other for the benchmark line: per configuration retrieve and inject
    microseconds, the injection's rate and its fraction of ``peak_gbs``, tokens injected and the sizes used.  A
    configuration that would start after ``budget_s`` seconds is reported as skipped."""
    import time

    out, t0 = {}, time.perf_counter()
    for name in names:
        if time.perf_counter() - t0 > budget_s:
            out[name] = {"skipped": f"time budget of {budget_s:.0f} s used up by the configurations before it"}
            continue
        t1 = time.perf_counter()
        try:
            ln = measure(name, iters, seed, want_pool_blocks=CONFIGURED_POOL_BLOCKS.get(name))
        except Exception as ex:  # a configuration that does not fit this box must not lose the whole line
            out[name] = {"error": str(ex)[:300]}
            torch.cuda.empty_cache()
            continue
        out[name] = {
            "retrieve_us": ln["retrieve_us"], "retrieve_back_to_back_us": ln["retrieve_back_to_back_us"],
            "retrieve_inject_call_us": ln["retrieve_inject_call_us"],
            "retrieve_emb_gbs": ln["retrieve_emb_gbs"], "inject_us": ln["inject_us"], "inject_gbs": ln["inject_gbs"],
            "frac_of_measured": ln["inject_gbs"] / peak_gbs, "tokens": ln["tokens_injected"], "us_per_request": ln["us_per_request"],
            "sizes_used": {"facts": ln["facts_scanned"], "resident_facts": ln["resident_facts"], "store_gib": round(ln["store_gib"], 2),
                           "pool_blocks": ln["pool_blocks"], "pool_gib": round(ln["pool_gib"], 2), "queries": ln["queries_per_call"],
                           "k": ln["k"], "k_injected": ln["k_injected"], "note": ln["sizes_note"]},
            "kernel_timeouts": ln["kernel_timeouts"], "wall_s": round(time.perf_counter() - t1, 1),
        }  # fmt: skip
    return out


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="users100")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--hot-per-user", type=int, default=None)
    ap.add_argument("--pool-blocks", type=int, default=None)
    ap.add_argument("--retrieve-only", action="store_true", help="embedding-only store, time the batched retrieval alone")
    ap.add_argument("--compose-cache", action="store_true", help="Llama shape, host-tier store: a repeated request with and without the composition cache")
    ap.add_argument("--host-tier", action="store_true", help="Llama shape with all K/V in the pinned host arena: inject over PCIe")
    ap.add_argument("--variants", action="store_true", help="Llama shape: bf16 cache, e4m3 cache, partial rotary (inject only)")
    ap.add_argument("--ann", type=int, default=0, metavar="ROWS", help="graph index on ROWS structured embedding rows")
    ap.add_argument("--permuted-chunks", action="store_true", help="Llama shape: 64-token chunks in random order, 1K-32K tokens")
    a = ap.parse_args()
    if a.permuted_chunks:
        for ln in measure_permuted_chunks(a.iters, a.seed):
            print(json.dumps(ln))
    elif a.ann:
        for ln in measure_ann(a.ann, a.iters, a.seed):
            print(json.dumps(ln))
    elif a.variants:
        for ln in measure_variants(a.iters, a.seed):
            print(json.dumps(ln))
    elif a.compose_cache:
        for ln in measure_compose_cache(a.iters, a.seed):
            print(json.dumps(ln))
    elif a.host_tier:
        for ln in measure_host_tier(a.iters, a.seed):
            print(json.dumps(ln))
    elif a.retrieve_only:
        print(json.dumps(measure_retrieve_only(a.config, a.iters, a.seed)))
    else:
        print(json.dumps(measure(a.config, a.iters, a.seed, a.hot_per_user, a.pool_blocks)))
