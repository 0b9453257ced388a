"""Helpers shared by the GPU parity tests: build a store from seeded inputs, and compare the CUDA
library's outputs with the CPU oracle under the acceptance rules:

  * fact ids: rank by rank the oracle's score of the GPU's id and of the oracle's id differ by < 1e-5
    (scores compared as fp32), no duplicates, all ids valid; without such a near-tie the lists are equal;
  * slots and V: bit-exact; every slot the oracle does not write still holds the sentinel;
  * K: |gpu - ref| <= 2^-7 * max(|ref|, 2^-10 * ||pair||) for every element, ref in double precision
    (outputs a thousand times smaller than their 2-d pair's norm are cancellation results, for which an
    error relative to the output itself is not attainable in fp32 arithmetic), and, wherever
    |ref| >= 2^-10 * ||pair||, at most 1 bf16 ulp away from the correctly rounded value.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2607_27090_b200 import synth
from paper_2607_27090_b200.memstore import MemStore, PagedCache

K_REL_TOL = 2.0**-7
K_FLOOR = 2.0**-10
SCORE_TIE = 1e-5


def to_dev(a: np.ndarray, device="cuda"):
    """numpy -> device tensor; uint16 arrays are bf16 bit patterns."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy bit patterns (host); a uint8 tensor (8-bit cache) -> its bytes."""
    if t.dtype == torch.uint8:
        return t.contiguous().cpu().numpy()
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class HostStore:
    """Seeded store kept on the host as well (small cases): lens, offs, k, v (uint16 [L, T, H, D]), emb."""

    def __init__(self, seed, n_facts, L, H, D, lo, hi, emb_dim, emb_dtype, n_users=1, lens=None):
        self.L, self.H, self.D = L, H, D
        self.n_users, self.per_user = n_users, n_facts
        total = n_facts * n_users
        self.lens = synth.fact_lengths(seed, total, lo, hi) if lens is None else np.asarray(lens, np.int32)
        self.offs = np.concatenate([[0], np.cumsum(self.lens)[:-1]]).astype(np.int64)
        T = int(self.lens.sum())
        self.k = np.empty((L, T, H, D), np.uint16)
        self.v = np.empty((L, T, H, D), np.uint16)
        for f in range(total):
            kf, vf = synth.kv_fact(seed, f, L, int(self.lens[f]), H, D)
            self.k[:, self.offs[f] : self.offs[f] + self.lens[f]] = kf
            self.v[:, self.offs[f] : self.offs[f] + self.lens[f]] = vf
        self.emb = synth.embeddings(seed, total, emb_dim, emb_dtype)
        self.emb_dim, self.emb_dtype = emb_dim, emb_dtype

    def to_memstore(self, theta, batch=64, extra_kv_tokens=0, **kw) -> MemStore:
        """Facts are added user by user in id order (ids are global and dense in insertion order)."""
        tdt = torch.float32 if self.emb_dtype == "float32" else torch.float16
        T = int(self.lens.sum())
        ms = MemStore(n_layers=self.L, n_kv_heads=self.H, head_dim=self.D, emb_dim=self.emb_dim, emb_dtype=tdt,
                      rope_theta=theta, n_users=self.n_users, max_facts_per_user=max(self.per_user, 1),
                      max_kv_tokens=max(T + extra_kv_tokens, 1), **kw)  # fmt: skip
        for u in range(self.n_users):
            for a in range(u * self.per_user, (u + 1) * self.per_user, batch):
                b = min((u + 1) * self.per_user, a + batch)
                t0, t1 = int(self.offs[a]), int(self.offs[b - 1] + self.lens[b - 1])
                first = ms.add_facts(to_dev(self.emb[a:b]), self.lens[a:b], to_dev(self.k[:, t0:t1]), to_dev(self.v[:, t0:t1]), user=u)
                assert first == a
        torch.cuda.synchronize()
        return ms


def check_ids(gpu_ids, gpu_scores, emb, query, k, row_ids=None, removed=None):
    """Near-tie rule for one query. ``emb``: the rows visible to the query; row_ids: their fact ids; removed: boolean per
    row, rows that must never be returned."""
    n = emb.shape[0]
    ids_o, sc_o = oracle.retrieve(emb, query, k, row_ids=row_ids, removed=removed)
    ids_o, sc_o = ids_o[0], sc_o[0]
    gpu_ids = np.asarray(gpu_ids)
    take = min(n if removed is None else int(n - np.count_nonzero(removed)), k)
    assert np.all(gpu_ids[take:] == -1), "padding must be -1"
    g = gpu_ids[:take]
    assert len(set(g.tolist())) == take, "duplicate ids"
    if row_ids is None:
        rows = g.astype(np.int64)
        assert np.all((g >= 0) & (g < n)), "invalid id"
    else:
        lookup = {int(f): i for i, f in enumerate(row_ids)}
        assert all(int(x) in lookup for x in g), "id outside the user's segment"
        rows = np.array([lookup[int(x)] for x in g], dtype=np.int64)
    if removed is not None:
        assert not np.asarray(removed)[rows].any(), "a removed fact was returned"
    # the oracle's exact score of every row the GPU chose
    s_gpu_choice = oracle.scores(emb[rows], query).astype(np.float32) if take else np.zeros(0, np.float32)
    diff = np.abs(s_gpu_choice - sc_o[:take])
    assert np.all(diff < SCORE_TIE), f"rank-wise score gap {diff.max()} (not a near-tie)"
    exact = g == ids_o[:take]  # ranks where the lists differ are swaps inside a near-tie group
    if gpu_scores is not None:
        gs = np.asarray(gpu_scores)
        assert np.all(np.abs(gs[:take] - s_gpu_choice) < 2e-6 + 1e-6 * np.abs(s_gpu_choice)), "fp32 score too far from the exact one"
        assert np.all(gs[take:] == 0)
    return int((~exact).sum())


ANN_MARGIN = 1e-6  # decisions of a graph search wider than this cannot depend on how a binary32 sum was ordered


def check_ann_search(ids, scores, counters, emb, graph, queries, k, removed=None, row_ids=None, **params):
    """Graph search of the CUDA library against the oracle, query by query.  The reference is the oracle's search over
    its double-precision scores: when every decision of that search was wider than ANN_MARGIN the GPU must return the
    same rows after the same number of steps and scored rows, with scores within binary32 accumulation error of the
    exact ones.  Only a query with a closer decision is compared with the oracle's binary32 lane-order search (which
    restates the kernels' summation order), bit for bit.  Returns (queries judged by the exact search, queries)."""
    ids, scores = np.asarray(ids), np.asarray(scores)
    exact = oracle.ann_search(emb, graph, queries, k, exact=True, removed=removed, **params)
    to_ids = (lambda r: r) if row_ids is None else (lambda r: np.where(r >= 0, np.asarray(row_ids)[np.maximum(r, 0)], -1))
    on_exact_side = 0
    for i in range(len(queries)):
        if exact.margin[i] > ANN_MARGIN:
            on_exact_side += 1
            assert np.array_equal(ids[i], to_ids(exact.ids[i])), (i, params)
            assert np.all(np.abs(scores[i] - exact.scores[i]) < 2e-6 + 1e-6 * np.abs(exact.scores[i])), (i, params)
            if counters is not None:
                assert counters[i, 0] == exact.iters[i] and counters[i, 1] == exact.scored[i], (i, params)
        else:
            lanes = oracle.ann_search(emb, graph, queries[i : i + 1], k, removed=removed, **params)
            assert np.array_equal(ids[i], to_ids(lanes.ids[0])), (i, params)
            assert np.array_equal(scores[i].view(np.uint32), lanes.scores[0].view(np.uint32)), (i, params)
            if counters is not None:
                assert counters[i, 0] == lanes.iters[0] and counters[i, 1] == lanes.scored[0], (i, params)
    return on_exact_side, len(queries)


def k_tolerance(k_ref: np.ndarray, style: int, rotary_dim: int = 0) -> np.ndarray:
    """Per-element tolerance 2^-7 * max(|ref|, 2^-10 * ||pair||); rotation preserves the pair norm.
    Coordinates beyond ``rotary_dim`` are copies: their "pair" is the element itself."""
    D = k_ref.shape[-1]
    R = rotary_dim or D
    lead = k_ref[..., :R]
    if style == 0:
        a, b = lead[..., : R // 2], lead[..., R // 2 :]
        nrm = np.sqrt(a * a + b * b)
        pair = np.concatenate([nrm, nrm], axis=-1)
    else:
        a, b = lead[..., 0::2], lead[..., 1::2]
        nrm = np.sqrt(a * a + b * b)
        pair = np.repeat(nrm, 2, axis=-1)
    pair = np.concatenate([pair, np.abs(k_ref[..., R:])], axis=-1)
    return K_REL_TOL * np.maximum(np.abs(k_ref), K_FLOOR * pair), pair


def check_k_fp8(gpu_codes: np.ndarray, want: np.ndarray, k_ref: np.ndarray, k_scale: float, style: int = 0, rotary_dim: int = 0):
    """Keys of an 8-bit (e4m3) cache against the oracle's codes ``want`` = code(bf16(ref) / scale) and its unrounded
    rotated keys ``k_ref``.  The code is a function of the bf16 key, so the only freedom is the one the bf16 path has:
    a rotated coordinate whose exact value lies within fp32 evaluation error (4e-6 of the pair norm) of a bf16
    rounding tie may have been rounded to the other neighbour, and then carries that neighbour's code.  Everything
    else, and every coordinate beyond ``rotary_dim`` (a copy), must carry exactly the oracle's code.
    Returns the fraction of codes equal to the oracle's."""
    _, pair = k_tolerance(k_ref, style, rotary_dim)
    slack = 4e-6 * pair
    assert not np.isnan(oracle.e4m3_to_double(gpu_codes)).any(), "NaN code in the cache"
    eq = gpu_codes == want
    if rotary_dim:
        assert np.all(eq[..., rotary_dim:]), "unrotated coordinates must carry exactly the oracle's code"
    below = oracle.e4m3_from_scaled_bf16(oracle.bf16_from_double(k_ref - slack), k_scale)
    above = oracle.e4m3_from_scaled_bf16(oracle.bf16_from_double(k_ref + slack), k_scale)
    assert np.all(eq | (gpu_codes == below) | (gpu_codes == above)), "wrong e4m3 code away from a bf16 rounding tie"
    return float(eq.mean()) if eq.size else 1.0


def check_k(gpu_bits: np.ndarray, k_ref: np.ndarray, style: int = 0, rotary_dim: int = 0):
    """Returns (fraction bit-equal to the correctly rounded value, worst error / tolerance)."""
    got = oracle.bf16_to_double(gpu_bits)
    tol, pair = k_tolerance(k_ref, style, rotary_dim)
    err = np.abs(got - k_ref)
    ratio = err / np.maximum(tol, 1e-300)
    worst = float(ratio.max()) if ratio.size else 0.0
    assert worst <= 1.0, f"K error {worst:.3f}x the tolerance"
    rounded = oracle.bf16_from_double(k_ref)
    eq = gpu_bits == rounded
    # 1-ulp rule away from cancellation: neighbouring bf16 bit patterns of the same sign differ by 1
    big = np.abs(k_ref) >= K_FLOOR * pair
    ulp_dist = np.abs(gpu_bits.astype(np.int32) - rounded.astype(np.int32))
    assert np.all(ulp_dist[big & ~eq] <= 1), "more than 1 bf16 ulp from the correctly rounded key"
    return float(eq.mean()) if eq.size else 1.0, worst


def gather_cache_rows(cache: PagedCache, slots: np.ndarray, layers=None):
    """Read rows at `slots` back from the device cache -> (k_bits, v_bits) [nl, m, H, D] uint16."""
    L = cache.k.shape[0]
    l0, l1 = (0, L) if layers is None else layers
    bs = cache.block_size
    sl = torch.from_numpy(np.asarray(slots, dtype=np.int64)).to(cache.k.device)
    blk, inb = sl // bs, sl % bs
    nhd = cache.layout == "NHD"  # [L][blocks][bs][H][D]
    out = []
    for t in (cache.k, cache.v):
        x = t[l0:l1]
        # advanced indices split by a slice put the indexed dimension first: [m, nl, H, D] -> [nl, m, H, D]
        rows = x[:, blk, inb] if nhd else x[:, blk, :, inb].permute(1, 0, 2, 3)
        out.append(bits(rows))
    return out


def untouched_mask_ok(cache: PagedCache, written_slots: np.ndarray, sentinel_bits: int) -> bool:
    """True iff every slot NOT in written_slots still holds the sentinel in every layer, head and plane."""
    bs = cache.block_size
    dev = cache.k.device
    keep = torch.ones(cache.num_blocks * bs, dtype=torch.bool, device=dev)
    if len(written_slots):
        keep[torch.from_numpy(np.asarray(written_slots, dtype=np.int64)).to(dev)] = False
    keep = keep.view(cache.num_blocks, bs)
    nhd = cache.layout == "NHD"
    fp8 = cache.k.dtype == torch.uint8  # then the sentinel is a byte
    sent = sentinel_bits if fp8 else (sentinel_bits - 0x10000 if sentinel_bits >= 0x8000 else sentinel_bits)
    for t in (cache.k, cache.v):
        for l in range(t.shape[0]):
            xl = t[l] if fp8 else (t[l].view(torch.int16) if t[l].is_contiguous() else t[l].contiguous().view(torch.int16))
            ok = xl == sent  # [blocks, bs, H, D] or [blocks, H, bs, D]
            ok = ok.all(dim=-1)
            ok = ok.all(dim=2) if nhd else ok.all(dim=1)  # -> [blocks, bs]
            if not bool(ok[keep].all()):
                return False
    return True


def with_prefix(hs: HostStore, placed, prefix):
    """The oracle's view of an injection that starts with the instruction prefix: the prefix (k, v uint16
    [L, n, H, D]) becomes one more fact after the store's own and leads the placement list."""
    pk, pv = prefix
    n = len(hs.lens)
    offs = np.concatenate([hs.offs, [int(hs.lens.sum())]]).astype(np.int64)
    lens = np.concatenate([hs.lens, [pk.shape[1]]]).astype(np.int32)
    k = np.concatenate([hs.k, pk], axis=1)
    v = np.concatenate([hs.v, pv], axis=1)
    return np.concatenate([[n], np.asarray(placed, np.int32)]).astype(np.int32), offs, lens, k, v


def run_inject_and_check(ms: MemStore, hs: HostStore, ids_np, start, table_np, cache: PagedCache, theta, style=0,
                         inv_freq=None, flags=0, sentinel=synth.SENTINEL_BF16, check_untouched=True, prefix=None,
                         rotary_dim=0, expect_status=0):  # fmt: skip
    """One request: inject on the GPU, run the oracle on the same ids, compare. Returns stats dict.
    ``prefix``: (k, v) of the instruction prefix the store holds, when ``flags`` asks for it."""
    dev = cache.k.device
    ids = torch.from_numpy(np.asarray(ids_np, np.int32).reshape(1, -1)).to(dev)
    sp = torch.tensor([start], dtype=torch.int32, device=dev)
    bt = torch.from_numpy(np.asarray(table_np, np.int32).reshape(1, -1)).to(dev)
    placed = np.asarray(ids_np, np.int32).reshape(-1)
    if flags & 1:
        placed = placed[::-1]
    offs, lens, hk, hv = hs.offs, hs.lens, hs.k, hs.v
    if flags & 2:
        placed, offs, lens, hk, hv = with_prefix(hs, placed, prefix)
    fp8 = cache.k.dtype == torch.uint8
    res = oracle.inject(placed, offs, lens, hk, hv, theta, start, table_np, cache.block_size,
                        cache.num_blocks, style=style, inv_freq_override=inv_freq, rotary_dim=rotary_dim,
                        k_scale=cache.k_scale if fp8 else None, v_scale=cache.v_scale if fp8 else None)  # fmt: skip
    slot_map = torch.full((1, max(res.m, 1) + 3), -7, dtype=torch.int64, device=dev)
    n_tok, status = ms.inject(ids, sp, bt, cache, out_slot_mapping=slot_map, flags=flags)
    torch.cuda.synchronize()
    assert int(status[0]) == expect_status, f"status {int(status[0])}"
    assert int(n_tok[0]) == res.m
    sm = slot_map[0].cpu().numpy()
    assert np.array_equal(sm[: res.m], res.slots) and np.all(sm[res.m :] == -7)
    out = {"m": res.m, "exact_frac": 1.0, "worst": 0.0}
    if res.m and fp8:
        kb, vb = gather_cache_rows(cache, res.slots)
        assert np.array_equal(vb, res.v_fp8), "V codes must be bit-exact (fp32 division, one rounding)"
        out["exact_frac"] = check_k_fp8(kb, res.k_fp8, res.k_ref, cache.k_scale, style, rotary_dim)
    elif res.m:
        kb, vb = gather_cache_rows(cache, res.slots)
        assert np.array_equal(vb, res.v), "V must be bit-exact"
        out["exact_frac"], out["worst"] = check_k(kb, res.k_ref, style, rotary_dim)
        if rotary_dim:
            assert np.array_equal(kb[..., rotary_dim:], res.k_bf16[..., rotary_dim:]), "coordinates beyond rotary_dim are copies"
    if check_untouched:
        assert untouched_mask_ok(cache, res.slots, sentinel), "a slot outside the request was modified"
    return out
