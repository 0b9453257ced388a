"""Pins for the oracle's composition + paged placement (CPU only).

The joint-prefill reference below is an independent formulation: it concatenates the selected facts into
one sequence and rotates it at positions p..p+m-1 with explicit rotation matrices (Theorem 2: a chunk
injected at offset v0 receives the keys a joint prefill would rotate at v0..v0+c-1), then places rows by
the page formula with plain Python integer arithmetic.
"""
import math
from pathlib import Path

import numpy as np
import pytest

from paper_2607_27090_b200 import synth

from test_oracle_rope import rotation_matrix

GOLDEN = Path(__file__).parent / "golden"


def make_store(oracle_mod, seed, n_facts, L, H, D, lo, hi):
    lens = synth.fact_lengths(seed, n_facts, lo, hi)
    offs = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    T = int(lens.sum())
    k = np.empty((L, T, H, D), np.uint16)
    v = np.empty((L, T, H, D), np.uint16)
    for f in range(n_facts):
        kf, vf = synth.kv_fact(seed, f, L, int(lens[f]), H, D)
        k[:, offs[f] : offs[f] + lens[f]] = kf
        v[:, offs[f] : offs[f] + lens[f]] = vf
    return lens, offs, k, v


def joint_prefill_reference(oracle_mod, ids, lens, offs, k, theta, start, style=0, inv_freq=None):
    """Concatenate, then rotate the whole sequence jointly with explicit matrices. Returns [L, m, H, D] float64."""
    L, _, H, D = k.shape
    seq = np.concatenate([k[:, offs[f] : offs[f] + lens[f]] for f in ids if f >= 0], axis=1)
    x = oracle_mod.bf16_to_double(seq)
    f32 = oracle_mod.inv_freq(D, theta) if inv_freq is None else inv_freq
    out = np.empty_like(x)
    for t in range(x.shape[1]):
        R = rotation_matrix(D, start + t, f32, style)
        out[:, t] = x[:, t] @ R.T
    return out


@pytest.mark.parametrize("start,bs,style", [(0, 16, 0), (16, 16, 0), (13, 16, 1), (4096, 32, 0), (5, 4, 0)])
def test_chunked_rope_equals_joint_prefill_and_page_formula(oracle_mod, start, bs, style):
    L, H, D, theta = 2, 2, 32, 1.0e4
    lens, offs, k, v = make_store(oracle_mod, 11, 12, L, H, D, 1, 9)
    ids = np.array([7, 2, 2, -1, 11, 0], dtype=np.int32)  # a repeat and a skipped entry
    m = int(sum(lens[i] for i in ids if i >= 0))
    n_table = (start + m + bs - 1) // bs
    num_blocks = n_table + 5
    table = synth.block_tables(1, num_blocks, n_table, 1)[0]
    res = oracle_mod.inject(ids, offs, lens, k, v, theta, start, table, bs, num_blocks, style=style)
    assert res.m == m
    # rotated keys == joint prefill of the concatenated sequence
    ref = joint_prefill_reference(oracle_mod, ids, lens, offs, k, theta, start, style)
    assert np.allclose(res.k_ref, ref, rtol=0, atol=1e-12)
    # bf16 output is the double result rounded once
    assert np.array_equal(res.k_bf16, oracle_mod.bf16_from_double(res.k_ref))
    # V rows are bit copies of the stored rows, in composed order
    vseq = np.concatenate([v[:, offs[f] : offs[f] + lens[f]] for f in ids if f >= 0], axis=1)
    assert np.array_equal(res.v, vseq)
    # slots: block_table[pos // bs] * bs + pos % bs, with Python integers
    want = [int(table[(start + t) // bs]) * bs + (start + t) % bs for t in range(m)]
    assert res.slots.tolist() == want and len(set(want)) == m


def test_cumulative_offsets_single_fact_and_k1(oracle_mod):
    L, H, D, theta, bs = 1, 1, 16, 1.0e4, 16
    lens, offs, k, v = make_store(oracle_mod, 12, 6, L, H, D, 3, 20)
    table = np.arange(64, dtype=np.int32)
    # single fact at an unaligned start crossing block boundaries
    f = int(np.argmax(lens))
    res = oracle_mod.inject([f], offs, lens, k, v, theta, 13, table, bs, 64)
    assert res.m == lens[f] and res.slots.tolist() == list(range(13, 13 + lens[f]))
    # fact i of a request starts at b_i = sum of the lengths before it: rotating fact i ALONE at
    # start + b_i gives the same keys as its slice of the composed segment
    ids = [3, 0, 5, 1]
    full = oracle_mod.inject(ids, offs, lens, k, v, theta, 7, table, bs, 64)
    b = 0
    for i in ids:
        alone = oracle_mod.inject([i], offs, lens, k, v, theta, 7 + b, table, bs, 64)
        assert np.array_equal(alone.k_ref, full.k_ref[:, b : b + lens[i]])
        assert alone.slots.tolist() == full.slots[b : b + lens[i]].tolist()
        b += int(lens[i])
    assert full.m == b
    # empty request and all-skipped request
    assert oracle_mod.inject([], offs, lens, k, v, theta, 0, table, bs, 64).m == 0
    assert oracle_mod.inject([-1, -1], offs, lens, k, v, theta, 0, table, bs, 64).m == 0


def test_position_zero_token_is_bit_identical_to_stored_key(oracle_mod):
    lens, offs, k, v = make_store(oracle_mod, 13, 4, 2, 2, 64, 4, 8)
    res = oracle_mod.inject([2], offs, lens, k, v, 5.0e5, 0, np.arange(4, dtype=np.int32), 16, 4)
    assert np.array_equal(res.k_bf16[:, 0], k[:, offs[2]])
    assert not np.array_equal(res.k_bf16[:, 1], k[:, offs[2] + 1])


def test_cache_image_identity_table_equals_composed_segment_and_rest_untouched(oracle_mod):
    L, H, D, bs, nb = 2, 2, 32, 16, 10
    lens, offs, k, v = make_store(oracle_mod, 14, 8, L, H, D, 5, 30)
    ids, start = [1, 6, 3], 16
    # separate K and V planes, layout [L][blocks][bs][H][D]
    strides = (nb * bs * H * D, bs * H * D, H * D, D)
    kc = np.full(L * nb * bs * H * D, synth.SENTINEL_BF16, np.uint16)
    vc = kc.copy()
    table = np.arange(nb, dtype=np.int32)
    res = oracle_mod.inject(ids, offs, lens, k, v, 1.0e4, start, table, bs, nb, k_cache=kc, v_cache=vc, cache_strides=strides)
    kc = kc.reshape(L, nb * bs, H, D)
    vc = vc.reshape(L, nb * bs, H, D)
    m = res.m
    assert np.array_equal(kc[:, start : start + m], res.k_bf16) and np.array_equal(vc[:, start : start + m], res.v)
    assert np.all(kc[:, :start] == synth.SENTINEL_BF16) and np.all(kc[:, start + m :] == synth.SENTINEL_BF16)
    assert np.all(vc[:, :start] == synth.SENTINEL_BF16) and np.all(vc[:, start + m :] == synth.SENTINEL_BF16)
    # shuffled table, stacked planes (K at plane 0, V at plane 1 of one buffer), head-major blocks
    table = synth.block_tables(3, nb, nb, 1)[0]
    buf = np.full(2 * L * nb * H * bs * D, synth.SENTINEL_BF16, np.uint16)
    plane = L * nb * H * bs * D
    strides = (nb * H * bs * D, H * bs * D, D, bs * D)  # [L][blocks][H][bs][D]
    res2 = oracle_mod.inject(ids, offs, lens, k, v, 1.0e4, start, table, bs, nb, k_cache=buf[:plane], v_cache=buf[plane:], cache_strides=strides)
    kc2 = buf[:plane].reshape(L, nb, H, bs, D)
    vc2 = buf[plane:].reshape(L, nb, H, bs, D)
    touched = np.zeros((nb, bs), bool)
    for t in range(m):
        blk, inb = divmod(int(res2.slots[t]), bs)
        touched[blk, inb] = True
    for t in range(m):
        pos = start + t
        blk, inb = int(table[pos // bs]), pos % bs
        assert np.array_equal(kc2[:, blk, :, inb], res.k_bf16[:, t]) and np.array_equal(vc2[:, blk, :, inb], res.v[:, t])
    untouched = ~touched
    assert np.all(kc2.transpose(1, 3, 0, 2, 4)[untouched] == synth.SENTINEL_BF16)
    assert np.all(vc2.transpose(1, 3, 0, 2, 4)[untouched] == synth.SENTINEL_BF16)


def test_attention_over_injected_cache_equals_attention_over_joint_prefill(oracle_mod):
    # the end-to-end meaning of the path: softmax(q K^T / sqrt(d)) V read back THROUGH the block table
    # equals the same attention over the jointly rotated, contiguous sequence
    L, H, D, bs, nb, theta, start = 1, 1, 32, 8, 12, 1.0e4, 5
    lens, offs, k, v = make_store(oracle_mod, 15, 5, L, H, D, 4, 12)
    ids = [4, 0, 2]
    table = synth.block_tables(4, nb, nb, 1)[0]
    strides = (nb * bs * H * D, bs * H * D, H * D, D)
    kc = np.zeros(L * nb * bs * H * D, np.uint16)
    vc = np.zeros_like(kc)
    res = oracle_mod.inject(ids, offs, lens, k, v, theta, start, table, bs, nb, k_cache=kc, v_cache=vc, cache_strides=strides)
    m = res.m
    kc = oracle_mod.bf16_to_double(kc).reshape(nb, bs, D)
    vc = oracle_mod.bf16_to_double(vc).reshape(nb, bs, D)
    q = np.random.default_rng(0).standard_normal(D)
    qN = oracle_mod.rope_rows(q[None], start + m, theta)[0]
    rows = [(int(table[(start + t) // bs]), (start + t) % bs) for t in range(m)]
    K = np.stack([kc[b, i] for b, i in rows])
    V = np.stack([vc[b, i] for b, i in rows])
    w = np.exp(K @ qN / math.sqrt(D))
    out_cache = (w / w.sum()) @ V
    Kj = joint_prefill_reference(oracle_mod, ids, lens, offs, k, theta, start)[0, :, 0]
    Vj = oracle_mod.bf16_to_double(np.concatenate([v[0, offs[f] : offs[f] + lens[f], 0] for f in ids]))
    w = np.exp(Kj @ qN / math.sqrt(D))
    out_joint = (w / w.sum()) @ Vj
    # only the single bf16 rounding of K separates the two
    assert np.allclose(out_cache, out_joint, rtol=0, atol=2e-2)
    Kj_b = oracle_mod.bf16_to_double(oracle_mod.bf16_from_double(Kj))
    w = np.exp(Kj_b @ qN / math.sqrt(D))
    assert np.allclose(out_cache, (w / w.sum()) @ Vj, rtol=0, atol=1e-12)


def test_inv_freq_override_and_layer_range(oracle_mod):
    L, H, D = 3, 2, 16
    lens, offs, k, v = make_store(oracle_mod, 16, 4, L, H, D, 2, 6)
    f = (np.arange(D // 2, dtype=np.float32) + 1) * 0.125
    table = np.arange(8, dtype=np.int32)
    full = oracle_mod.inject([1, 3], offs, lens, k, v, 1.0e4, 3, table, 8, 8, inv_freq_override=f)
    ref = joint_prefill_reference(oracle_mod, [1, 3], lens, offs, k, 1.0e4, 3, inv_freq=f)
    assert np.allclose(full.k_ref, ref, atol=1e-12)
    part = oracle_mod.inject([1, 3], offs, lens, k, v, 1.0e4, 3, table, 8, 8, inv_freq_override=f, layers=(1, 3))
    assert np.array_equal(part.k_ref, full.k_ref[1:3]) and np.array_equal(part.v, full.v[1:3])


def test_errors(oracle_mod):
    lens, offs, k, v = make_store(oracle_mod, 17, 3, 1, 1, 16, 4, 4)
    t = np.arange(2, dtype=np.int32)
    with pytest.raises(oracle_mod.OracleError) as e:
        oracle_mod.inject([0, 1, 2], offs, lens, k, v, 1e4, 0, t, 4, 2)  # 12 tokens need 3 blocks
    assert e.value.code == oracle_mod.ERR_BLOCK_TABLE
    with pytest.raises(oracle_mod.OracleError) as e:
        oracle_mod.inject([0], offs, lens, k, v, 1e4, 0, np.array([5], np.int32), 4, 2)
    assert e.value.code == oracle_mod.ERR_BLOCK_ID


def test_storage_cost_matches_paper_figure(oracle_mod):
    for line in (GOLDEN / "storage_cost.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        L, c, h, d, b, want = (int(x) for x in line.split())
        assert oracle_mod.kv_bytes(L, c, h, d, b) == want
    assert synth.CONFIGS["llama8b"].token_bytes == 131072
