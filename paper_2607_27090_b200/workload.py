"""Builds the seeded synthetic workloads (``synth.CONFIGS``) on one GPU: a populated ``MemStore``, a paged
cache pool, queries and block tables.  Used by the benchmark and by the full-size parity tests.

Only input generation and calls into the binding happen here; no step of the method is computed in Python.
K/V values are drawn on the device per fact from (seed, fact id), so a fact can be redrawn later (for the
CPU oracle) without keeping a second copy of a store that is tens of GiB.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import synth
from .memstore import MemStore, PagedCache


@dataclass
class Workload:
    shape: synth.Shape
    seed: int
    store: MemStore
    lens: np.ndarray  # [n_users * n_facts] tokens per fact (0: embedding-only)
    emb: np.ndarray  # host copy of all embeddings [n_users * n_facts, E]
    queries: np.ndarray  # host [nq_pool, E]
    cache: PagedCache | None
    device: torch.device

    def fact_kv_host(self, fact_id: int):
        """Redraw one fact's K_pre and V on the device and return them as uint16 bit patterns on the host."""
        s = self.shape
        k, v = synth.kv_fact_device(self.seed, fact_id, s.n_layers, int(self.lens[fact_id]), s.n_kv_heads, s.head_dim, self.device)
        f = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)  # noqa: E731
        return f(k), f(v)

    def host_pack(self, fact_ids):
        """Host arrays for the oracle holding only the given facts: (offsets, lengths, k, v) where offsets and
        lengths are indexed by GLOBAL fact id (other facts have length 0 and must not be referenced)."""
        s = self.shape
        uniq = sorted({int(f) for f in fact_ids if f >= 0})
        lens = np.zeros(self.lens.size, np.int32)
        offs = np.zeros(self.lens.size, np.int64)
        T = int(sum(self.lens[f] for f in uniq))
        k = np.empty((s.n_layers, T, s.n_kv_heads, s.head_dim), np.uint16)
        v = np.empty_like(k)
        t = 0
        for f in uniq:
            n = int(self.lens[f])
            kf, vf = self.fact_kv_host(f)
            k[:, t : t + n], v[:, t : t + n] = kf, vf
            lens[f], offs[f] = n, t
            t += n
        return offs, lens, k, v


def build(name: str, seed: int = 0, device="cuda", n_query_pool: int | None = None, num_blocks: int | None = None,
          resident_ids=None, hot_per_user: int | None = None, scale_facts: float = 1.0, add_batch_tokens: int = 4096,
          want_cache: bool = True, emb: np.ndarray | None = None, queries: np.ndarray | None = None) -> Workload:  # fmt: skip
    """Create the store of configuration ``name`` and fill it.

    ``resident_ids``: for configurations with a hot subset, the global fact ids that must have K/V (the
    harness passes the ids its requests will inject); random filler ids complete the subset up to
    ``hot_per_user`` facts per user (default: the configuration's figure).
    ``scale_facts`` < 1 shrinks the number of facts per user (tests on smaller boxes).
    ``emb`` / ``queries``: arrays already drawn with ``synth.embeddings`` / ``synth.queries`` for the same seed
    (saves drawing a million rows twice)."""
    s = synth.CONFIGS[name]
    dev = torch.device(device)
    n_per_user = max(1, int(round(s.n_facts * scale_facts)))
    total = n_per_user * s.n_users
    lens = synth.fact_lengths(seed, total, s.len_lo, s.len_hi)
    if s.resident_per_user is not None:
        hot = np.zeros(total, bool)
        if resident_ids is not None:
            hot[np.asarray(sorted({int(i) for i in resident_ids if i >= 0}), np.int64)] = True
        rng = np.random.default_rng([seed, 6])
        per_user_hot = hot_per_user if hot_per_user is not None else max(1, int(round(s.resident_per_user * scale_facts)))
        for u in range(s.n_users):
            seg = np.arange(u * n_per_user, (u + 1) * n_per_user)
            missing = per_user_hot - int(hot[seg].sum())
            if missing > 0:
                cold = seg[~hot[seg]]
                hot[rng.choice(cold, size=min(missing, cold.size), replace=False)] = True
        lens = np.where(hot, lens, 0).astype(np.int32)
    if emb is None:
        emb = synth.embeddings(seed, total, s.emb_dim, s.emb_dtype)
    nq_pool = n_query_pool or max(s.nq, 16)
    if queries is None:
        queries = synth.queries(seed, nq_pool, s.emb_dim, s.emb_dtype)
    assert emb.shape == (total, s.emb_dim) and queries.shape[1] == s.emb_dim
    tdt = torch.float32 if s.emb_dtype == "float32" else torch.float16
    store = MemStore(device=dev.index or 0, n_layers=s.n_layers, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim,
                     emb_dim=s.emb_dim, emb_dtype=tdt, rope_theta=s.rope_theta, n_users=s.n_users,
                     max_facts_per_user=n_per_user, max_kv_tokens=max(1, int(lens.sum())))  # fmt: skip
    # add facts user by user, in id order, in batches bounded by tokens (staging buffers stay small)
    for u in range(s.n_users):
        a = u * n_per_user
        end = (u + 1) * n_per_user
        while a < end:
            b, tok = a, 0
            while b < end and (b == a or tok + lens[b] <= add_batch_tokens) and b - a < 65536:
                tok += int(lens[b])
                b += 1
            ks, vs = [], []
            for f in range(a, b):
                if lens[f]:
                    k, v = synth.kv_fact_device(seed, f, s.n_layers, int(lens[f]), s.n_kv_heads, s.head_dim, dev)
                    ks.append(k)
                    vs.append(v)
            k_pack = torch.cat(ks, dim=1).contiguous() if ks else None
            v_pack = torch.cat(vs, dim=1).contiguous() if vs else None
            e = torch.from_numpy(emb[a:b]).to(dev)
            first = store.add_facts(e, lens[a:b], k_pack, v_pack, user=u)
            assert first == a
            a = b
    torch.cuda.synchronize(dev)
    cache = None
    if want_cache:
        nb = num_blocks or default_num_blocks(s)
        cache = PagedCache.allocate(s.n_layers, nb, s.block_size, s.n_kv_heads, s.head_dim, dev)
    return Workload(s, seed, store, lens, emb, queries, cache, dev)


def default_num_blocks(s: synth.Shape) -> int:
    per_req = blocks_per_request(s, s.k)
    return max(1024, 1 << int(np.ceil(np.log2(per_req * max(16, s.nq)))))


def blocks_per_request(s: synth.Shape, k: int) -> int:
    """Block-table length that covers the prefix plus k facts of the maximum length."""
    return (s.start_pos + k * s.len_hi + s.block_size - 1) // s.block_size


def kv_bytes_moved(s: synth.Shape, m_tokens: int) -> int:
    """Algorithmic bytes of injecting m tokens: unrotated K and V read once, rotated K and V written once."""
    return 2 * m_tokens * s.token_bytes


def emb_bytes_scanned(s: synth.Shape, n_rows: int) -> int:
    return n_rows * s.emb_dim * (4 if s.emb_dtype == "float32" else 2)
