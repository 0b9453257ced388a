"""GPU parity tests of the graph index: the beam search against the oracle's search over double-precision scores (same
rows, steps and row counts wherever that search's closest decision is wider than binary32 rounding; the rest bit for bit
against the oracle's binary32 lane-order search), the graph build against the oracle's exact neighbour graph (near-tie rule of the exact
retrieval), recall against exact retrieval on structured rows, and the error paths."""
import numpy as np
import pytest
import torch

from paper_2607_27090_b200 import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import oracle
    from parity import check_ann_search, to_dev
    from paper_2607_27090_b200.memstore import MemStore, MemStoreError

DEV = "cuda"


def emb_store(emb, n_users=1):
    n, E = emb.shape
    ms = MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=E, emb_dtype=torch.float32 if emb.dtype == np.float32 else torch.float16,
                  rope_theta=1e4, n_users=n_users, max_facts_per_user=max(n, 1), max_kv_tokens=0)  # fmt: skip
    for a in range(0, n, 50_000):
        b = min(n, a + 50_000)
        ms.add_facts(to_dev(emb[a:b]), np.zeros(b - a, np.int32))
    return ms


@pytest.mark.parametrize("dtype,dim,n,deg,kind", [
    ("float32", 64, 3000, 16, "knn"), ("float16", 1024, 2000, 64, "random"), ("float16", 136, 5000, 8, "random"),
    ("float16", 256, 700, 32, "knn"), ("float32", 8, 40, 4, "random"),
])  # fmt: skip
def test_search_equals_the_oracle(dtype, dim, n, deg, kind):
    emb = synth.embeddings_low_rank(80, n, dim, dtype, intrinsic_dim=min(8, dim))
    emb[n // 2] = emb[3]  # equal scores: the lower row goes first
    graph = oracle.knn_graph(emb, deg) if kind == "knn" else synth.random_graph(81, n, deg)
    if kind == "random":
        graph[5, 0] = n + 7  # a row outside the segment is ignored
    q = synth.queries_near_rows(82, emb, 9)
    q[0] = emb[3]
    ms = emb_store(emb)
    ms.set_graph(to_dev(graph))
    assert torch.equal(ms.get_graph().cpu(), torch.from_numpy(graph))
    judged_exact = judged = 0
    for k, beam, parents, n_entry, max_iters in ((10, 64, 4, 64, 32), (1, 1, 1, 1, 50), (50, 16, 2, 7, 5), (100, 128, 8, 200, 12),
                                                  (256, 256, 1, 512, 3)):  # fmt: skip
        if parents * deg > 512:
            continue
        par = dict(beam=beam, parents=parents, n_entry=n_entry, max_iters=max_iters)
        ids, sc, cnt = ms.retrieve_ann(to_dev(q), k, want_counters=True, **par)
        torch.cuda.synchronize()
        a, b = check_ann_search(ids.cpu().numpy(), sc.cpu().numpy(), cnt.cpu().numpy(), emb, graph, q, k, **par)
        judged_exact, judged = judged_exact + a, judged + b
    # most searches are decided by margins that no binary32 summation order can overturn: those are judged against the
    # double-precision search alone
    print(f"graph search parity: {judged_exact} of {judged} queries judged by the exact search")
    assert judged_exact >= 0.75 * judged
    # the scores are those of the exact path
    ids, sc = ms.retrieve_ann(to_dev(q), 5)
    ex_ids, ex_sc = ms.retrieve(to_dev(q), n if n < 100 else 100)
    for i in range(len(q)):
        lookup = dict(zip(ex_ids[i].tolist(), ex_sc[i].tolist()))
        assert all(lookup.get(a, b) == b for a, b in zip(ids[i].tolist(), sc[i].tolist()))
    ms.close()


@pytest.mark.parametrize("dtype,dim,n,deg", [("float32", 64, 2500, 16), ("float16", 128, 9000, 64), ("float16", 64, 30, 40), ("float32", 32, 8500, 12)])
def test_graph_build_matches_the_exact_neighbour_graph(dtype, dim, n, deg):
    """Rows as queries through the exact retrieval kernels (CUDA-core path below 8193 rows, tensor-core filter
    above); compared with the oracle's graph under the near-tie rule of exact retrieval."""
    emb = synth.embeddings_low_rank(83, n, dim, dtype, intrinsic_dim=min(8, dim))
    for r in (7, 11, 19):
        emb[r] = emb[2]  # four identical rows
    ms = emb_store(emb)
    ms.build_graph(deg)
    g = ms.get_graph().cpu().numpy()
    assert g.shape == (n, deg)
    want = oracle.knn_graph(emb, deg)
    rows = list(range(0, n, max(1, n // 40))) + [2, 7, 11, 19, n - 1]
    exact_same = 0
    for r in rows:
        got = g[r]
        valid = got[got >= 0]
        assert len(valid) == min(deg, n - 1) and np.all(got[len(valid):] == -1)
        assert r not in valid and len(set(valid.tolist())) == len(valid) and np.all(valid < n)
        s_got = oracle.scores(emb[valid], emb[r])
        s_want = oracle.scores(emb[want[r][: len(valid)]], emb[r])
        assert np.all(np.abs(s_got.astype(np.float32) - s_want.astype(np.float32)) < 1e-5)
        exact_same += int(np.array_equal(valid, want[r][: len(valid)]))
    assert exact_same >= len(rows) * 0.8
    assert set(g[2][:3].tolist()) == {7, 11, 19} and g[7][0] == 2
    ms.close()


def test_recall_against_exact_retrieval_on_structured_rows():
    n, dim, k = 60_000, 128, 10
    emb = synth.embeddings_low_rank(84, n, dim, "float16", intrinsic_dim=16)
    q = synth.queries_near_rows(85, emb, 48)
    ms = emb_store(emb)
    ms.build_graph(32)
    ex_ids, _ = ms.retrieve(to_dev(q), k)
    recalls = {}
    for beam in (16, 64, 128):
        ids, _, cnt = ms.retrieve_ann(to_dev(q), k, beam=beam, want_counters=True)
        a, b = ids.cpu().numpy(), ex_ids.cpu().numpy()
        recalls[beam] = float(np.mean([len(set(a[i]) & set(b[i])) / k for i in range(len(q))]))
        assert int(cnt[:, 1].max()) < n // 4  # far fewer rows scored than a scan
    assert recalls[64] >= 0.9 and recalls[128] >= recalls[16]
    # the library's graph, handed to the oracle, gives the oracle the same answers (search parity at this size)
    g = ms.get_graph().cpu().numpy()
    ids, sc = ms.retrieve_ann(to_dev(q[:6]), k)
    check_ann_search(ids.cpu().numpy(), sc.cpu().numpy(), None, emb, g, q[:6], k, beam=64, parents=8, n_entry=64, max_iters=32)  # the library's defaults at degree 32
    ms.close()


def test_graph_search_with_removed_rows():
    """Removed rows stay in the graph: the walk goes through them and the result passes them over (the oracle's rule)."""
    n, dim, deg = 4000, 128, 16
    emb = synth.embeddings_low_rank(94, n, dim, "float16", intrinsic_dim=8)
    q = synth.queries_near_rows(95, emb, 10)
    ms = emb_store(emb)
    ms.build_graph(deg)
    g = ms.get_graph().cpu().numpy()
    removed = np.random.default_rng(94).random(n) < 0.15
    first, _ = ms.retrieve_ann(to_dev(q), 5)
    removed[first[:, 0].cpu().numpy()] = True  # every query loses its best row
    for f in np.flatnonzero(removed):
        ms.remove_fact(int(f))
    for k, beam in ((10, 64), (50, 64), (64, 64), (100, 128)):
        par = dict(beam=beam, parents=4, n_entry=64, max_iters=32)
        ids, sc, cnt = ms.retrieve_ann(to_dev(q), k, want_counters=True, **par)
        torch.cuda.synchronize()
        ids_np = ids.cpu().numpy()
        assert not np.isin(ids_np[ids_np >= 0], np.flatnonzero(removed)).any()
        check_ann_search(ids_np, sc.cpu().numpy(), cnt.cpu().numpy(), emb, g, q, k, removed=removed, **par)
    # a graph built now lists no removed row
    ms.build_graph(deg)
    g2 = ms.get_graph().cpu().numpy()
    assert not np.isin(g2, np.flatnonzero(removed)).any()
    ms.close()


@pytest.mark.parametrize("dtype,dim,per_user,n_users,deg", [("float16", 128, 400, 5, 16), ("float32", 64, 152, 3, 8)])
def test_every_user_segment_has_its_own_graph(dtype, dim, per_user, n_users, deg):
    """Graphs of a multi-user store: built per segment (rows local to the segment), searched for the query's user,
    results are that user's fact ids; appended rows are linked per user; a caller-made graph can be set per user."""
    total = per_user * n_users
    emb = synth.embeddings_low_rank(96, total, dim, dtype, intrinsic_dim=6)
    tdt = torch.float32 if dtype == "float32" else torch.float16
    ms = MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=dim, emb_dtype=tdt, rope_theta=1e4, n_users=n_users,
                  max_facts_per_user=per_user + 40, max_kv_tokens=0)  # fmt: skip
    # facts arrive interleaved: ids are global, rows are per segment
    row_ids = [[] for _ in range(n_users)]
    nxt = 0
    for chunk in range(4):
        for u in range(n_users):
            a = u * per_user + chunk * (per_user // 4)
            b = a + per_user // 4
            first = ms.add_facts(to_dev(emb[a:b]), np.zeros(b - a, np.int32), user=u)
            assert first == nxt
            row_ids[u].extend(range(nxt, nxt + (b - a)))
            nxt += b - a
    ms.build_graph(deg)
    users = np.array([u % n_users for u in range(2 * n_users)], np.int32)
    q = np.stack([synth.queries_near_rows(97 + i, emb[u * per_user : (u + 1) * per_user], 1)[0] for i, u in enumerate(users)])
    par = dict(beam=64, parents=4, n_entry=32, max_iters=20)
    graphs = []
    for u in range(n_users):
        seg = emb[u * per_user : (u + 1) * per_user]
        g = ms.get_graph(user=u).cpu().numpy()
        assert g.shape == (per_user, deg) and g.max() < per_user
        want = oracle.knn_graph(seg, deg)
        same = 0
        for r in range(0, per_user, 7):
            s_got = oracle.scores(seg[g[r]], seg[r]).astype(np.float32)
            s_want = oracle.scores(seg[want[r]], seg[r]).astype(np.float32)
            assert np.all(np.abs(s_got - s_want) < 1e-5) and r not in g[r]
            same += int(np.array_equal(g[r], want[r]))
        assert same >= 0.8 * len(range(0, per_user, 7))
        graphs.append(g)
    ids, sc, cnt = ms.retrieve_ann(to_dev(q), 10, want_counters=True, query_users=to_dev(users), **par)
    torch.cuda.synchronize()
    for i, u in enumerate(users):
        seg = emb[u * per_user : (u + 1) * per_user]
        check_ann_search(ids[i : i + 1].cpu().numpy(), sc[i : i + 1].cpu().numpy(), cnt[i : i + 1].cpu().numpy(), seg, graphs[u], q[i : i + 1], 10,
                         row_ids=np.array(row_ids[u], np.int32), **par)
    # exact and approximate retrieval agree on the best fact of a query that is a stored row
    probe = emb[2 * per_user + 5 : 2 * per_user + 6]
    ids_a, _ = ms.retrieve_ann(to_dev(probe), 1, query_users=to_dev(np.array([2], np.int32)))
    ids_e, _ = ms.retrieve(to_dev(probe), 1, query_users=to_dev(np.array([2], np.int32)))
    assert int(ids_a[0, 0]) == int(ids_e[0, 0]) == row_ids[2][5]
    # rows appended to two segments are linked into those segments' graphs
    extra = synth.embeddings_low_rank(98, 40, dim, dtype, intrinsic_dim=6)
    ms.add_facts(to_dev(extra[:25]), np.zeros(25, np.int32), user=1)
    ms.add_facts(to_dev(extra[25:]), np.zeros(15, np.int32), user=n_users - 1)
    ms.graph_append()
    assert ms.get_graph(user=1).shape == (per_user + 25, deg) and ms.get_graph(user=0).shape == (per_user, deg)
    seg1 = np.concatenate([emb[per_user : 2 * per_user], extra[:25]])
    want1 = oracle.graph_append(seg1, oracle.knn_graph(seg1[:per_user], deg))
    g1 = ms.get_graph(user=1).cpu().numpy()
    for r in list(range(per_user, per_user + 25)) + list(range(0, per_user, 11)):
        s_got = oracle.scores(seg1[g1[r]], seg1[r]).astype(np.float32)
        s_want = oracle.scores(seg1[want1[r]], seg1[r]).astype(np.float32)
        assert np.all(np.abs(s_got - s_want) < 1e-5), r
    # a caller-made graph for one user replaces that user's graph only
    custom = synth.random_graph(99, per_user, deg)
    ms.set_graph(to_dev(custom), user=0)
    assert torch.equal(ms.get_graph(user=0).cpu(), torch.from_numpy(custom)) and ms.get_graph(user=1).shape[0] == per_user + 25
    ids_c, sc_c = ms.retrieve_ann(to_dev(q[:1]), 5, query_users=to_dev(users[:1]), **par)
    check_ann_search(ids_c.cpu().numpy(), sc_c.cpu().numpy(), None, emb[:per_user], custom, q[:1], 5, row_ids=np.array(row_ids[0], np.int32), **par)
    ms.close()


def test_graph_index_errors_and_empty_cases():
    emb = synth.embeddings(86, 100, 64, "float16")
    ms = emb_store(emb)
    q = to_dev(synth.queries(86, 2, 64, "float16"))
    with pytest.raises(MemStoreError):  # no graph yet
        ms.retrieve_ann(q, 5)
    ms.build_graph(8)
    for bad in (dict(beam=300), dict(parents=33), dict(parents=8, n_entry=513), dict(max_iters=100000)):
        with pytest.raises(MemStoreError):
            ms.retrieve_ann(q, 5, **bad)
    with pytest.raises(MemStoreError):
        ms.retrieve_ann(q, 300)
    with pytest.raises(MemStoreError):
        ms.build_graph(0)
    with pytest.raises(MemStoreError):
        ms.set_graph(torch.zeros((101, 4), dtype=torch.int32, device=DEV))  # more rows than facts
    ids, _ = ms.retrieve_ann(q, 5)  # still usable after the refused calls
    assert bool((ids >= 0).all())
    ms.close()
    with pytest.raises(MemStoreError):
        ms_bad = emb_store(emb[:50])
        ms_bad.set_graph(torch.zeros((10, 4), dtype=torch.int32, device=DEV), user=1)  # no such user
    empty = MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=64, rope_theta=1e4, max_facts_per_user=10, max_kv_tokens=0)
    empty.build_graph(4)
    ids, sc = empty.retrieve_ann(q, 3)
    assert ids.cpu().tolist() == [[-1] * 3] * 2 and sc.cpu().tolist() == [[0.0] * 3] * 2
    empty.close()


def test_measurement_modes_of_the_package_run_at_small_sizes():
    """The committed measurement entry points (graph index, cache variants, retrieval alone) keep working: run them
    at toy sizes and check that their lines are sane."""
    from paper_2607_27090_b200 import measure_configs as mc

    lines = mc.measure_ann(20_000, 2, dim=128, degree=16, k=10, intrinsic_dim=8)
    assert len(lines) == 3 and all(ln["recall_at_k"] > 0.8 and ln["ann_us_1_query"] > 0 for ln in lines)
    lines = mc.measure_variants(2, n_facts=60, k=10)
    assert [ln["config"].split()[1] for ln in lines] == ["bf16", "e4m3", "rotary_dim"]
    assert lines[1]["bytes_moved"] == 0.75 * lines[0]["bytes_moved"] and all(ln["inject_us"] > 0 for ln in lines)
    line = mc.measure_retrieve_only("tiny", 2)
    assert line["kernel_timeouts"] == 0 and line["retrieve_us"] > 0


def test_retrieve_inject_through_the_graph_index():
    """MS_RETRIEVE_ANN: index search, then planning and the copy kernel, in one call and from host buffers; the cache
    is the one that retrieve_ann followed by inject gives, and memstore_inject itself refuses the flag."""
    from parity import HostStore
    from paper_2607_27090_b200 import memstore as M
    from paper_2607_27090_b200.memstore import PagedCache

    hs = HostStore(87, 300, 2, 4, 64, 4, 20, 64, "float16")
    hs.emb = synth.embeddings_low_rank(87, 300, 64, "float16", intrinsic_dim=6)
    ms = hs.to_memstore(1e4)
    ms.build_graph(16)
    bs, nb, k = 16, 128, 8
    q = synth.queries_near_rows(88, hs.emb, 3)
    starts = to_dev(np.array([0, 5, 17], np.int32))
    tables = to_dev(synth.block_tables(89, nb, 16, 3))
    ca = PagedCache.allocate(hs.L, nb, bs, hs.H, hs.D, DEV, fill_bits=synth.SENTINEL_BF16)
    cb = PagedCache.allocate(hs.L, nb, bs, hs.H, hs.D, DEV, fill_bits=synth.SENTINEL_BF16)
    ids_a, _ = ms.retrieve_ann(to_dev(q), k)
    n_a, st_a = ms.inject(ids_a, starts, tables, ca, flags=M.INJECT_REVERSE)
    ids_b, n_b, st_b = ms.retrieve_inject(to_dev(q), k, starts, tables, cb, flags=M.INJECT_REVERSE | M.RETRIEVE_ANN)
    torch.cuda.synchronize()
    assert torch.equal(ids_a, ids_b) and torch.equal(n_a, n_b) and int(st_b.abs().sum()) == 0
    assert torch.equal(ca.k.view(torch.int16), cb.k.view(torch.int16)) and torch.equal(ca.v.view(torch.int16), cb.v.view(torch.int16))
    ids_s, sc_s = ms.retrieve_ann(to_dev(q), k)
    assert torch.equal(ids_s, ids_b)
    check_ann_search(ids_s.cpu().numpy(), sc_s.cpu().numpy(), None, hs.emb, ms.get_graph().cpu().numpy(), q, k, beam=64, parents=8, n_entry=64, max_iters=32)
    out = np.full(k + 2, -5, np.int32)
    cc = PagedCache.allocate(hs.L, nb, bs, hs.H, hs.D, DEV, fill_bits=synth.SENTINEL_BF16)
    ms.serve_host(q[1], k, 5, tables[1].cpu().numpy(), cc, out, flags=M.INJECT_REVERSE | M.RETRIEVE_ANN)
    assert out[:k].tolist() == ids_b[1].cpu().tolist() and out[k] == int(n_b[1]) and out[k + 1] == 0
    with pytest.raises(MemStoreError):
        ms.inject(ids_a, starts, tables, ca, flags=M.RETRIEVE_ANN)
    ms.close()


@pytest.mark.parametrize("dtype,dim,n_old,n_add,deg", [("float32", 32, 900, 150, 8), ("float16", 128, 9000, 200, 64), ("float16", 64, 0, 90, 16),
                                                       ("float16", 64, 500, 70, 100)])  # fmt: skip
def test_graph_append_matches_the_oracle_rule(dtype, dim, n_old, n_add, deg):
    """Rows added after the build are linked by memstore_graph_append: their own lists are exact, and an old row keeps
    the best of its list plus the new rows that list it.  Compared row by row with the oracle's graph (its own build,
    its own append) under the near-tie rule; then the grown graph is searched."""
    n = n_old + n_add
    emb = synth.embeddings_low_rank(93, n, dim, dtype, intrinsic_dim=min(6, dim))
    ms = MemStore(n_layers=1, n_kv_heads=1, head_dim=16, emb_dim=dim, emb_dtype=torch.float32 if dtype == "float32" else torch.float16,
                  rope_theta=1e4, max_facts_per_user=n, max_kv_tokens=0)  # fmt: skip
    if n_old:
        ms.add_facts(to_dev(emb[:n_old]), np.zeros(n_old, np.int32))
    ms.build_graph(deg)
    ms.graph_append()  # nothing added yet: a no-op
    assert ms.get_graph().shape == (n_old, deg)
    for a in range(n_old, n, 64):  # facts arrive in several calls
        b = min(n, a + 64)
        ms.add_facts(to_dev(emb[a:b]), np.zeros(b - a, np.int32))
    ms.graph_append()
    g = ms.get_graph().cpu().numpy()
    assert g.shape == (n, deg)
    want = oracle.graph_append(emb, oracle.knn_graph(emb[:n_old], deg) if n_old else np.zeros((0, deg), np.int32))
    rows = list(range(0, n, max(1, n // 60))) + list(range(n_old, n, 7)) + [n - 1]
    changed = [r for r in range(n_old) if not np.array_equal(want[r], oracle.knn_graph(emb[:n_old], deg)[r])] if n_old and n_old <= 1000 else []
    rows += changed[:40]
    same = 0
    for r in rows:
        got = g[r][g[r] >= 0]
        exp = want[r][want[r] >= 0]
        assert len(got) == len(exp) == min(deg, n - 1) and r not in got and len(set(got.tolist())) == len(got)
        s_got = oracle.scores(emb[got], emb[r]).astype(np.float32)
        s_exp = oracle.scores(emb[exp], emb[r]).astype(np.float32)
        assert np.all(np.abs(s_got - s_exp) < 1e-5), r
        same += int(np.array_equal(got, exp))
    assert same >= 0.8 * len(rows)
    if n_old and n_old <= 1000:
        assert len(changed) > 10  # the append did change old rows' lists
    # the grown graph is searched like any other; new rows are found
    q = emb[n - 3 : n].copy()
    ids, _ = ms.retrieve_ann(to_dev(q), 5, beam=64)
    assert ids[:, 0].cpu().tolist() == [n - 3, n - 2, n - 1]
    ms.close()
