"""The allocation-free retrieve entry point (memstore_retrieve_static) against memstore_retrieve.

It serves callers that cannot let the library allocate device memory while they run: its scratch is a fixed
array inside the library.  This file is named so that pytest collects it last: if it fails, a run that stops at
the first failure has already run every other test.  It must pass alone in a fresh process and after the rest.
"""
import numpy as np
import pytest
import torch

from paper_2607_27090_b200 import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from parity import HostStore, check_ids, to_dev
    from paper_2607_27090_b200 import memstore as M
    from paper_2607_27090_b200.memstore import MemStore


def both(ms, q, k, users=None):
    """Same query batch through the allocating and the allocation-free entry points, outputs preallocated."""
    nq = q.shape[0]
    ids_a = torch.full((nq, k), -9, dtype=torch.int32, device="cuda")
    sc_a = torch.full((nq, k), -9.0, dtype=torch.float32, device="cuda")
    ids_b, sc_b = ids_a.clone(), sc_a.clone()
    ms.retrieve(q, k, query_users=users, out_ids=ids_a, out_scores=sc_a)
    ms.retrieve_static(q, k, query_users=users, out_ids=ids_b, out_scores=sc_b)
    torch.cuda.synchronize()
    return ids_a.cpu().numpy(), sc_a.cpu().numpy(), ids_b.cpu().numpy(), sc_b.cpu().numpy()


@pytest.mark.parametrize("n_facts,dtype,E", [(777, "float16", 1024), (300, "float32", 64), (9000, "float16", 128)])
def test_static_retrieve_matches_retrieve_on_two_calls_in_a_row(n_facts, dtype, E):
    # 9000 rows exceed the fused kernel's segment size, so the scores-then-top-k pair runs through the static scratch too
    hs = HostStore(21, n_facts, 1, 1, 16, 1, 2, E, dtype)
    ms = hs.to_memstore(1e4)
    q_all = synth.queries(21, 8, E, dtype)
    for call, (lo, hi, k) in enumerate([(0, 5, 50), (5, 8, 7)]):  # the second call sees the first call's leftovers
        q = to_dev(q_all[lo:hi])
        ids_a, sc_a, ids_b, sc_b = both(ms, q, k)
        assert np.array_equal(ids_a, ids_b), f"call {call}: ids differ"
        assert np.all(np.abs(sc_a - sc_b) <= 2e-6), f"call {call}: scores differ"
        for i in range(hi - lo):  # and both are right
            check_ids(ids_b[i], sc_b[i], hs.emb, q_all[lo + i], k)
    ms.close()


def test_static_retrieve_per_user_segments_and_shared_scratch_between_stores():
    hs1 = HostStore(22, 60, 1, 1, 16, 1, 2, 128, "float16", n_users=3)
    hs2 = HostStore(23, 200, 1, 1, 16, 1, 2, 128, "float16")
    ms1, ms2 = hs1.to_memstore(1e4), hs2.to_memstore(1e4)
    users = to_dev(np.array([2, 0, 1, 1], np.int32))
    q1, q2 = to_dev(synth.queries(22, 4, 128, "float16")), to_dev(synth.queries(23, 2, 128, "float16"))
    for _ in range(2):  # alternate stores: each call finds the other store's scores and tickets in the scratch
        a = both(ms1, q1, 12, users)
        assert np.array_equal(a[0], a[2]) and np.all(np.abs(a[1] - a[3]) <= 2e-6)
        b = both(ms2, q2, 30)
        assert np.array_equal(b[0], b[2]) and np.all(np.abs(b[1] - b[3]) <= 2e-6)
    ms1.close()
    ms2.close()


def test_static_retrieve_refuses_sizes_beyond_its_scratch():
    ms = MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=64, max_facts_per_user=(1 << 20) // 4 + 1, max_kv_tokens=1)
    q = to_dev(synth.queries(0, 4, 64, "float16"))
    with pytest.raises(M.MemStoreError) as e:
        ms.retrieve_static(q, 3)  # 4 queries x (2^18 + 1) rows > 2^20 scores
    assert e.value.code == 4 and "static scratch" in str(e.value)
    ids, _ = ms.retrieve_static(q[:3], 3)  # 3 x (2^18 + 1) fits; the store is empty
    assert torch.all(ids == -1)
    small = MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=64, max_facts_per_user=8, max_kv_tokens=1)
    with pytest.raises(M.MemStoreError) as e:
        small.retrieve_static(to_dev(synth.queries(0, 1025, 64, "float16")), 3)
    assert e.value.code == 4
    ms.close()
    small.close()
