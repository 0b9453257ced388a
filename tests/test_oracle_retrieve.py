"""Pins for the oracle's scoring and top-k (CPU only): numpy float64 matmul as the library routine,
a full sort, brute force on tiny inputs, and the special cases k = 1, k = N, k > N, empty store."""
import itertools

import numpy as np
import pytest

from paper_2607_27090_b200 import synth


@pytest.mark.parametrize("dtype", ["float32", "float16"])
def test_scores_equal_float64_matmul(oracle_mod, dtype):
    emb = synth.embeddings(0, 300, 64, dtype)
    q = synth.queries(0, 3, 64, dtype)
    ref = q.astype(np.float64) @ emb.astype(np.float64).T  # exact products, library summation
    for i in range(3):
        s = oracle_mod.scores(emb, q[i])
        assert np.allclose(s, ref[i], rtol=0, atol=1e-14)


def test_scores_hand_example(oracle_mod):
    emb = np.array([[1, 0, 0, 0], [0.5, 0.5, 0.5, 0.5], [0, -1, 0, 2], [0.25, 0, 0, 0]], dtype=np.float16)
    q = np.array([2, 4, -1, 0.5], dtype=np.float16)
    assert oracle_mod.scores(emb, q).tolist() == [2.0, 2.75, -3.0, 0.5]
    ids, sc = oracle_mod.retrieve(emb, q, 3)
    assert ids.tolist() == [[1, 0, 3]] and sc.tolist() == [[2.75, 2.0, 0.5]]


@pytest.mark.parametrize("dtype", ["float32", "float16"])
def test_topk_equals_full_sort(oracle_mod, dtype):
    n, e = 1000, 128
    emb = synth.embeddings(1, n, e, dtype)
    q = synth.queries(1, 4, e, dtype)
    s = q.astype(np.float64) @ emb.astype(np.float64).T
    for k in (1, 5, 100, n):
        ids, sc = oracle_mod.retrieve(emb, q, k)
        for i in range(4):
            order = np.lexsort((np.arange(n), -oracle_mod.scores(emb, q[i])))  # score desc, id asc
            assert np.array_equal(ids[i], order[:k])
            assert np.allclose(sc[i], s[i, order[:k]], rtol=0, atol=1e-7)
    ids, _ = oracle_mod.retrieve(emb, q, 1)
    assert np.array_equal(ids[:, 0], np.argmax(s, axis=1))  # k = 1 is the argmax


def test_topk_brute_force_tiny(oracle_mod):
    # tiny: every k-subset, pick the one with the largest total score; it must be the oracle's set
    rng = np.random.default_rng(2)
    emb = rng.standard_normal((9, 8)).astype(np.float32)
    q = rng.standard_normal(8).astype(np.float32)
    s = emb.astype(np.float64) @ q.astype(np.float64)
    for k in (1, 2, 4):
        best = max(itertools.combinations(range(9), k), key=lambda c: sum(s[list(c)]))
        ids, _ = oracle_mod.retrieve(emb, q, k)
        assert set(ids[0].tolist()) == set(best)
        assert np.all(np.diff(s[ids[0]]) <= 0)  # best first


def test_ties_go_to_lower_id_and_query_equal_to_a_row_ranks_first(oracle_mod):
    emb = synth.embeddings(3, 64, 32, "float16")
    emb[40] = emb[7]  # planted duplicates: identical scores
    emb[50] = emb[7]
    q = emb[7].copy()
    ids, sc = oracle_mod.retrieve(emb, q, 5)
    assert ids[0, :3].tolist() == [7, 40, 50]
    assert sc[0, 0] == pytest.approx(1.0, abs=2e-3) and sc[0, 0] == sc[0, 1] == sc[0, 2]
    # all-equal embeddings: ids come back in increasing order
    same = np.tile(emb[:1], (10, 1))
    ids, _ = oracle_mod.retrieve(same, q, 10)
    assert ids[0].tolist() == list(range(10))


def test_row_ids_map_rows_to_fact_ids(oracle_mod):
    emb = synth.embeddings(4, 20, 16, "float32")
    q = synth.queries(4, 1, 16, "float32")
    row_ids = np.arange(20, dtype=np.int32) * 3 + 100
    a, _ = oracle_mod.retrieve(emb, q, 6)
    b, _ = oracle_mod.retrieve(emb, q, 6, row_ids=row_ids)
    assert np.array_equal(b, a * 3 + 100)


def test_k_larger_than_store_and_empty_store(oracle_mod):
    emb = synth.embeddings(5, 3, 16, "float32")
    q = synth.queries(5, 2, 16, "float32")
    ids, sc = oracle_mod.retrieve(emb, q, 6)
    assert np.all(ids[:, 3:] == -1) and np.all(sc[:, 3:] == 0)
    assert all(sorted(r[:3].tolist()) == [0, 1, 2] for r in ids)
    ids, _ = oracle_mod.retrieve(np.zeros((0, 16), np.float32), q, 4)
    assert np.all(ids == -1)
