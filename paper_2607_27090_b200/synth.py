"""Seeded synthetic inputs shaped like the paper's memory-profile serving workload.

This module only DRAWS inputs (lengths, embeddings, queries, K/V values, block
tables).  It contains none of the method's arithmetic (no scoring, no top-k, no
rotation, no slot computation) and imports neither the CUDA binding nor the CPU
oracle, so both sides can be fed from it.

Shapes follow the evaluation set-up of the paper (Sec. 6.1): short facts, a
unit-norm embedding per fact searched by inner product, k between 5 and 100,
bf16 KV, 16-token cache pages, up to 100 concurrent users.  The paper's own
dataset is not available; these inputs stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# bf16 bit pattern used to pre-fill caches in tests (a finite value, -1.2109375e2, that a copy or
# rotation of N(0,1) data will not produce by accident in every element of a row)
SENTINEL_BF16 = 0xC2F2


@dataclass(frozen=True)
class Shape:
    """One workload configuration (names follow the paper: L layers, h KV heads, d head dim)."""

    name: str
    n_layers: int
    n_kv_heads: int
    head_dim: int
    rope_theta: float
    n_facts: int  # per user
    len_lo: int
    len_hi: int
    emb_dim: int
    emb_dtype: str  # "float32" | "float16"
    nq: int
    k: int
    block_size: int
    start_pos: int
    n_users: int = 1
    resident_per_user: int | None = None  # None: every fact has K/V in HBM
    ks: tuple = field(default=())

    @property
    def row_elems(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def token_bytes(self) -> int:
        """K+V bytes of one token over all layers: 2 * L * h * d * 2 (Sec. 3.5 with c = 1, bf16)."""
        return 2 * self.n_layers * self.row_elems * 2


CONFIGS = {
    "tiny": Shape("tiny", 1, 2, 64, 1.0e4, 256, 8, 32, 64, "float32", 1, 5, 16, 16),
    "llama8b": Shape("llama8b", 32, 8, 128, 5.0e5, 2000, 16, 64, 1024, "float16", 1, 50, 16, 32, ks=(5, 10, 20, 50)),
    "users100": Shape(
        "users100", 32, 8, 128, 5.0e5, 500, 16, 64, 1024, "float16", 100, 20, 16, 32, n_users=100, resident_per_user=40
    ),
    "gqa14b": Shape("gqa14b", 40, 8, 128, 1.0e6, 5000, 32, 128, 1024, "float16", 1, 100, 32, 4096),
    "stress1m": Shape(
        "stress1m", 32, 8, 128, 5.0e5, 1_000_000, 16, 64, 1024, "float16", 64, 100, 16, 32, resident_per_user=20_000
    ),
}


def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(s) for s in stream]])


def fact_lengths(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    """Integer token counts, uniform on [lo, hi], both ends included."""
    return _rng(seed, 1).integers(lo, hi + 1, size=n).astype(np.int32)


def unit_rows(seed: int, stream: int, n: int, dim: int, dtype: str, chunk: int = 65536) -> np.ndarray:
    """i.i.d. Gaussian rows, normalised to unit length in float32, then rounded to ``dtype`` (not re-normalised).
    Every chunk of rows has its own generator, so chunks are drawn in parallel threads with identical results."""
    out = np.empty((n, dim), dtype=np.dtype(dtype))

    def draw(c: int) -> None:
        a = c * chunk
        b = min(n, a + chunk)
        x = _rng(seed, stream, c).standard_normal((b - a, dim), dtype=np.float32)
        x /= np.linalg.norm(x, axis=1, keepdims=True)
        out[a:b] = x.astype(out.dtype)

    n_chunks = (n + chunk - 1) // chunk
    if n_chunks <= 1:
        for c in range(n_chunks):
            draw(c)
    else:
        from concurrent.futures import ThreadPoolExecutor
        import os

        with ThreadPoolExecutor(max_workers=min(n_chunks, os.cpu_count() or 1, 16)) as pool:
            list(pool.map(draw, range(n_chunks)))
    return out


def embeddings(seed: int, n: int, dim: int, dtype: str) -> np.ndarray:
    return unit_rows(seed, 2, n, dim, dtype)


def queries(seed: int, nq: int, dim: int, dtype: str) -> np.ndarray:
    return unit_rows(seed, 3, nq, dim, dtype)


def embeddings_low_rank(seed: int, n: int, dim: int, dtype: str, intrinsic_dim: int = 32, noise: float = 0.05,
                        chunk: int = 65536) -> np.ndarray:  # fmt: skip
    """Unit-norm rows with low intrinsic dimension, the structure that text embeddings have and isotropic Gaussian
    rows lack (on which no proximity graph can beat a full scan): a Gaussian latent vector of ``intrinsic_dim``
    coordinates goes through a fixed random linear map to ``dim`` coordinates, a little isotropic noise is added,
    and the row is normalised in float32 and rounded to ``dtype``."""
    proj = _rng(seed, 4).standard_normal((intrinsic_dim, dim)).astype(np.float32) / np.sqrt(intrinsic_dim)
    out = np.empty((n, dim), dtype=np.float32 if dtype == "float32" else np.float16)
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        g = _rng(seed, 5, a)
        z = g.standard_normal((b - a, intrinsic_dim)).astype(np.float32)
        x = z @ proj + noise * g.standard_normal((b - a, dim)).astype(np.float32)
        x /= np.linalg.norm(x, axis=1, keepdims=True)
        out[a:b] = x
    return out


def queries_near_rows(seed: int, emb: np.ndarray, nq: int, noise: float = 0.3) -> np.ndarray:
    """Queries that resemble stored rows: a random row plus isotropic noise of relative norm ``noise``, normalised."""
    g = _rng(seed, 6)
    rows = g.integers(0, emb.shape[0], nq)
    x = emb[rows].astype(np.float32)
    x += noise * g.standard_normal(x.shape).astype(np.float32) / np.sqrt(emb.shape[1])
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    return x.astype(emb.dtype)


def random_graph(seed: int, n: int, deg: int, holes: float = 0.05) -> np.ndarray:
    """A seeded directed graph as search input: ``deg`` random neighbours per row (repeats and self-loops
    allowed), a share ``holes`` of the entries set to -1, int32 [n, deg]."""
    g = _rng(seed, 7)
    out = g.integers(0, max(n, 1), (n, deg)).astype(np.int32)
    out[g.random((n, deg)) < holes] = -1
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def kv_fact(seed: int, fact_id: int, n_layers: int, n_tokens: int, n_heads: int, head_dim: int):
    """K_pre and V of one fact, N(0,1) rounded to bf16, as uint16 bit patterns [L, n_tokens, h, d]."""
    g = _rng(seed, 4, fact_id)
    shape = (n_layers, n_tokens, n_heads, head_dim)
    k = f32_to_bf16_bits(g.standard_normal(shape, dtype=np.float32))
    v = f32_to_bf16_bits(g.standard_normal(shape, dtype=np.float32))
    return k, v


def kv_fact_device(seed: int, fact_id: int, n_layers: int, n_tokens: int, n_heads: int, head_dim: int, device):
    """Device-side draw of one fact's K_pre and V (bf16 tensors).  Regenerable from (seed, fact_id) on the
    same device, so a large store needs no second copy: the harness redraws the facts it hands to the oracle."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1_000_003 + int(fact_id)) * 2 + 1)
    shape = (2, n_layers, n_tokens, n_heads, head_dim)
    kv = torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    return kv[0], kv[1]


def block_tables(seed: int, num_blocks: int, blocks_per_request: int, nreq: int) -> np.ndarray:
    """A random permutation of the block pool dealt out to the requests: distinct, non-contiguous blocks."""
    need = blocks_per_request * nreq
    if need > num_blocks:
        raise ValueError(f"{need} blocks needed, pool has {num_blocks}")
    perm = _rng(seed, 5).permutation(num_blocks)[:need].astype(np.int32)
    return perm.reshape(nreq, blocks_per_request)
