"""Pins for the oracle's graph index (CPU only): the exact neighbour graph and the beam search in its two forms - ranking by
the plain double-precision scores (the definition, with the margin of its closest decision) and ranking by binary32 sums
in one stated order (for cases decided inside binary32 rounding).  Each check is against something other than the
oracle's own code: exact sums with a rounding behaviour known by construction, numpy's float64 matmul and argsort,
brute force over all rows where the search must degenerate to it, walks on a path graph that can be followed by hand,
margins planted in the inputs, and agreement of the two forms wherever the margin exceeds binary32 rounding."""
import numpy as np
import pytest

from paper_2607_27090_b200 import synth


def test_f32_scores_follow_the_stated_lane_order(oracle_mod):
    # dim 512 in halves: 64 vectors of 8, vector v in lane v mod 32, two vectors per lane.
    # element 0 carries a product of 2^24; a further 1.0 added to 2^24 in binary32 is lost (ties to even).
    dim = 512
    row = np.zeros((1, dim), np.float16)
    q = np.ones(dim, np.float16)
    row[0, 0], q[0] = 4096.0, 4096.0
    row[0, 1:8] = 1.0  # same vector, same lane, added after the big product: all seven are lost
    assert oracle_mod.scores_f32(row, q)[0] == 2.0**24
    row[0, 256:264] = 1.0  # vector 32 is lane 0 again: lost as well
    assert oracle_mod.scores_f32(row, q)[0] == 2.0**24
    row[0, 8:16] = 1.0  # vector 1 is lane 1: its 8 is kept and joins in the butterfly
    assert oracle_mod.scores_f32(row, q)[0] == 2.0**24 + 8
    row[0, 1:8] = 0
    row[0, 256:264] = 0
    row[0, 8:16] = 0
    row[0, 504:512] = 0.5  # last vector (63) is lane 31: 8 * 0.5 = 4 survives
    assert oracle_mod.scores_f32(row, q)[0] == 2.0**24 + 4
    # float32 rows: vectors of 4 elements
    r32 = np.zeros((1, 256), np.float32)
    q32 = np.ones(256, np.float32)
    r32[0, 0] = 2.0**24
    r32[0, 1:4] = 1.0  # same vector as element 0
    r32[0, 128:132] = 1.0  # vector 32: lane 0 again
    r32[0, 4:8] = 1.0  # vector 1, lane 1
    assert oracle_mod.scores_f32(r32, q32)[0] == 2.0**24 + 4


def test_f32_scores_are_close_to_the_double_scores(oracle_mod):
    for dtype, dim in (("float16", 1024), ("float32", 64), ("float16", 136)):
        emb = synth.embeddings(1, 300, dim, dtype)
        q = synth.queries(1, 1, dim, dtype)[0]
        exact = oracle_mod.scores(emb, q)
        assert np.abs(oracle_mod.scores_f32(emb, q) - exact).max() < 3e-7


def test_knn_graph_against_numpy_argsort(oracle_mod):
    emb = synth.embeddings_low_rank(2, 400, 64, "float32", intrinsic_dim=8)
    emb[37] = emb[5]  # duplicate rows: equal scores against every third row, lower row first
    g = oracle_mod.knn_graph(emb, 10)
    s = emb.astype(np.float64) @ emb.astype(np.float64).T
    np.fill_diagonal(s, -np.inf)
    for r in (0, 5, 37, 399, 123):
        order = np.lexsort((np.arange(400), -s[r]))[:10]
        # numpy's pairwise summation differs from a left-to-right sum in the last bits: compare scores, not ids
        assert np.allclose(s[r][g[r]], s[r][order], rtol=0, atol=1e-12) and len(set(g[r].tolist())) == 10 and r not in g[r]
    assert g[5][0] == 37 and g[37][0] == 5
    both = [r for r in range(400) if 5 in g[r] and 37 in g[r]]
    assert both and all(list(g[r]).index(5) + 1 == list(g[r]).index(37) for r in both)  # tie: row 5 right before row 37
    tiny = oracle_mod.knn_graph(emb[:4], 6)
    assert np.all(tiny[:, 3:] == -1) and np.all(tiny[:, :3] >= 0)  # fewer rows than neighbours: padded


@pytest.mark.parametrize("exact", [False, True])
def test_search_on_a_complete_graph_is_brute_force(oracle_mod, exact):
    n, dim, k = 150, 64, 12
    emb = synth.embeddings(3, n, dim, "float32")
    complete = np.array([[c for c in range(n) if c != r] for r in range(n)], np.int32)
    q = synth.queries(3, 4, dim, "float32")
    res = oracle_mod.ann_search(emb, complete, q, k, beam=4, parents=1, n_entry=1, max_iters=3, exact=exact)
    want, want_sc = oracle_mod.retrieve(emb, q, k)
    assert np.array_equal(res.ids, want)
    assert np.all(res.scored == n) and np.all(res.iters >= 1)
    for i in range(4):
        if exact:  # the double scores rounded to binary32, as exact retrieval reports them
            assert np.array_equal(res.scores[i], want_sc[i])
        else:
            assert np.array_equal(res.scores[i], oracle_mod.scores_f32(emb, q[i])[res.ids[i]])


@pytest.mark.parametrize("exact", [False, True])
def test_search_with_a_beam_as_large_as_the_store_visits_the_whole_component(oracle_mod, exact):
    n, dim = 300, 64
    emb = synth.embeddings_low_rank(4, n, dim, "float32", intrinsic_dim=6)
    g = oracle_mod.knn_graph(emb, 8)
    q = synth.queries_near_rows(4, emb, 3)
    res = oracle_mod.ann_search(emb, g, q, 10, beam=n, parents=3, n_entry=n, max_iters=1000, exact=exact)
    want, _ = oracle_mod.retrieve(emb, q, 10)
    assert np.array_equal(res.ids, want) and np.all(res.scored == n)  # every row is an entry point here


def arc(n):
    a = np.linspace(0.0, 1.0, n)
    return np.stack([np.cos(a), np.sin(a)] + [np.zeros(n)] * 6, axis=1).astype(np.float32)  # dim 8


@pytest.mark.parametrize("exact", [False, True])
def test_greedy_walk_on_a_path_graph_can_be_followed_by_hand(oracle_mod, exact):
    # 100 points on an arc, row i linked to i-1 and i+1; the only entry point is (1 * 2654435761) mod 100 = 61.
    n = 100
    emb = arc(n)
    path = np.array([[i - 1 if i > 0 else -1, i + 1 if i + 1 < n else -1] for i in range(n)], np.int32)
    q = emb[70:71].copy()
    # beam 1: each step expands the single listed row and moves one row towards 70; 9 moves, then the step that
    # expands 70 itself finds nothing better; the next look finds no unexpanded entry
    res = oracle_mod.ann_search(emb, path, q, 1, beam=1, parents=1, n_entry=1, max_iters=50, exact=exact)
    # rows scored: the entry, 60 and 62 in step 1, then one new row per step (the other neighbour was seen): 63..70, 71
    assert res.ids[0, 0] == 70 and res.iters[0] == 10 and res.scored[0] == 1 + 2 + 8 + 1
    res = oracle_mod.ann_search(emb, path, q, 1, beam=1, parents=1, n_entry=1, max_iters=5, exact=exact)
    assert res.ids[0, 0] == 66 and res.iters[0] == 5
    # beam 3 keeps the trail: after 4 steps the list is 65, 64, 63 (closest to 70 first)
    res = oracle_mod.ann_search(emb, path, q, 3, beam=3, parents=1, n_entry=1, max_iters=4, exact=exact)
    assert res.ids[0].tolist() == [65, 64, 63]
    # two entry points, 61 and (2 * 2654435761) mod 100 = 22: the walk from 61 still wins, 22 is never expanded first
    res = oracle_mod.ann_search(emb, path, q, 2, beam=2, parents=1, n_entry=2, max_iters=50, exact=exact)
    assert res.ids[0].tolist() == [70, 71] or res.ids[0].tolist() == [70, 69]
    assert abs(float(res.scores[0, 0]) - 1.0) < 1e-6


@pytest.mark.parametrize("exact", [False, True])
def test_holes_bad_rows_padding_and_duplicate_entry_points(oracle_mod, exact):
    emb = arc(10)
    g = np.array([[-1, 11], [0, 2], [1, 1], [2, 2], [-5, 3], [4, 4], [5, 5], [6, 6], [7, 7], [8, 8]], np.int32)
    # entry (2654435761 mod 10) = 1; from 1 the walk reaches 0 and 2 only; rows 3.. point backwards
    res = oracle_mod.ann_search(emb, g, emb[9:10], 5, beam=5, parents=2, n_entry=1, max_iters=20, exact=exact)
    assert sorted(res.ids[0, :3].tolist()) == [0, 1, 2] and res.ids[0, 3:].tolist() == [-1, -1] and res.scored[0] == 3
    assert res.scores[0, 3:].tolist() == [0.0, 0.0]
    # 30 entry points on 10 rows: duplicates dropped, at most 10 rows scored
    res = oracle_mod.ann_search(emb, g, emb[9:10], 3, beam=3, parents=1, n_entry=30, max_iters=0, exact=exact)
    assert res.scored[0] <= 10 and res.iters[0] == 0 and res.ids[0, 0] >= 0
    # empty store
    res = oracle_mod.ann_search(emb[:0], g[:0], emb[9:10], 2, exact=exact)
    assert res.ids[0].tolist() == [-1, -1]
    if exact:
        assert res.margin[0] == np.inf  # nothing was ever compared


def test_decision_margin_is_the_gap_planted_in_the_inputs(oracle_mod):
    """Rows whose score against the query e_0 is their first coordinate, on a complete graph with every row an entry
    point: the list is the sorted scores, and the margin is the smallest gap between neighbours down to the cut."""
    vals = np.array([1.0, 0.5, 0.5 + 2.0**-20, 0.25, 0.125, 0.125 - 2.0**-12, -0.75, 0.0625], np.float32)
    n = len(vals)
    emb = np.zeros((n, 8), np.float32)
    emb[:, 0] = vals
    emb[:, 1] = np.arange(n)  # rows differ elsewhere too (orthogonal to the query)
    q = np.zeros((1, 8), np.float32)
    q[0, 0] = 1.0
    complete = np.array([[c for c in range(n) if c != r] for r in range(n)], np.int32)
    order = np.argsort(-vals.astype(np.float64), kind="stable")
    res = oracle_mod.ann_search(emb, complete, q, n, beam=n, parents=1, n_entry=n, max_iters=4, exact=True)
    assert res.ids[0].tolist() == order.tolist() and res.margin[0] == 2.0**-20
    # a cut at L = 3 still looks at the pair (kept 2, dropped 3) = (0.5, 0.25), and no further: the 2^-12 gap is below the cut
    res = oracle_mod.ann_search(emb, complete, q, 3, beam=3, parents=1, n_entry=n, max_iters=0, exact=True)
    assert res.ids[0].tolist() == order[:3].tolist() and res.margin[0] == 2.0**-20
    res = oracle_mod.ann_search(emb, complete, q, 1, beam=1, parents=1, n_entry=n, max_iters=0, exact=True)
    assert res.ids[0].tolist() == [0] and res.margin[0] == 1.0 - (0.5 + 2.0**-20)
    # identical rows tie in every arithmetic and are ordered by row: their pair is not a decision
    emb2 = emb.copy()
    emb2[3] = emb2[1]
    res = oracle_mod.ann_search(emb2, complete, q, n, beam=n, parents=1, n_entry=n, max_iters=4, exact=True)
    assert res.ids[0, :4].tolist() == [0, 2, 1, 3] and res.margin[0] == 2.0**-20
    # equal scores of rows that differ elsewhere: a decision with margin zero (any other arithmetic may order them otherwise)
    emb3 = emb.copy()
    emb3[3, 0] = emb3[1, 0]
    res = oracle_mod.ann_search(emb3, complete, q, n, beam=n, parents=1, n_entry=n, max_iters=4, exact=True)
    assert res.ids[0, :4].tolist() == [0, 2, 1, 3] and res.margin[0] == 0.0


def test_the_binary32_search_takes_the_exact_walk_wherever_the_margin_exceeds_its_rounding(oracle_mod):
    """The two forms share the walk's bookkeeping but not the arithmetic that ranks: wherever every decision of the
    exact search is wider than 1e-6 (binary32 sums of unit-norm rows are within 3e-7 of the exact ones) the lane-order
    search must return the same rows after the same steps.  A wrong lane order, a dropped vector or a mis-added partial
    sum moves scores by far more than that and breaks the agreement."""
    total = agree_needed = 0
    for seed, dtype, dim, n, deg in ((1, "float16", 1024, 1500, 32), (2, "float32", 64, 3000, 16), (3, "float16", 136, 2500, 8)):
        emb = synth.embeddings_low_rank(seed, n, dim, dtype, intrinsic_dim=8)
        g = oracle_mod.knn_graph(emb, deg) if seed != 3 else synth.random_graph(seed, n, deg)
        q = synth.queries_near_rows(seed + 10, emb, 12)
        for k, beam, parents, n_entry, max_iters in ((10, 64, 4, 64, 32), (50, 16, 2, 7, 5), (100, 128, 8, 200, 12)):
            a = oracle_mod.ann_search(emb, g, q, k, beam=beam, parents=parents, n_entry=n_entry, max_iters=max_iters)
            b = oracle_mod.ann_search(emb, g, q, k, beam=beam, parents=parents, n_entry=n_entry, max_iters=max_iters, exact=True)
            for i in range(len(q)):
                total += 1
                if b.margin[i] > 1e-6:
                    agree_needed += 1
                    assert np.array_equal(a.ids[i], b.ids[i]) and a.iters[i] == b.iters[i] and a.scored[i] == b.scored[i]
                    assert np.abs(a.scores[i] - b.scores[i]).max() < 3e-7
    assert agree_needed > 0.8 * total


def test_recall_grows_with_the_beam_on_structured_rows(oracle_mod):
    n, dim, k = 3000, 64, 10
    emb = synth.embeddings_low_rank(5, n, dim, "float32", intrinsic_dim=8)
    g = oracle_mod.knn_graph(emb, 16)
    q = synth.queries_near_rows(5, emb, 20)
    want, _ = oracle_mod.retrieve(emb, q, k)

    def recall(beam):
        got = oracle_mod.ann_search(emb, g, q, k, beam=beam, parents=2, n_entry=16, max_iters=200).ids
        return np.mean([len(set(got[i]) & set(want[i])) / k for i in range(len(q))])

    r_small, r_large = recall(10), recall(96)
    assert r_large >= r_small and r_large > 0.9


def test_graph_append_rule(oracle_mod):
    n_old, n, dim, deg = 300, 360, 32, 8
    emb = synth.embeddings_low_rank(6, n, dim, "float32", intrinsic_dim=5)
    old = oracle_mod.knn_graph(emb[:n_old], deg)
    new = oracle_mod.graph_append(emb, old)
    full = oracle_mod.knn_graph(emb, deg)
    # new rows: the exact lists of a fresh graph
    assert np.array_equal(new[n_old:], full[n_old:])
    s = emb.astype(np.float64) @ emb.astype(np.float64).T
    touched = 0
    for nb in range(n_old):
        offers = [r for r in range(n_old, n) if nb in new[r]]
        if not offers:
            assert np.array_equal(new[nb], old[nb])  # nobody offered anything
            continue
        touched += 1
        pool = np.array(list(old[nb]) + offers)
        order = pool[np.lexsort((pool, -s[nb][pool]))][:deg]  # brute force with numpy: best deg of old list + offers
        assert np.allclose(s[nb][new[nb]], s[nb][order], rtol=0, atol=1e-12)
        assert np.all(s[nb][new[nb]] >= s[nb][old[nb]] - 1e-12)  # a list only improves, entry by entry
        assert len(set(new[nb].tolist())) == deg and nb not in new[nb]
    assert touched > 20
    # appending in two steps is appending at once when the first step's rows are fixed... for the OLD rows' lists:
    half = oracle_mod.graph_append(emb[: n_old + 30], old)
    both = oracle_mod.graph_append(emb, half)
    # rows of the first step were given lists over 330 rows only, so compare the old rows offered by second-step rows
    for nb in range(n_old):
        offers_all = {r for r in range(n_old, n) if nb in new[r]}
        offers_two = {r for r in range(n_old, n_old + 30) if nb in half[r]} | {r for r in range(n_old + 30, n) if nb in both[r]}
        if offers_all == offers_two:
            assert np.array_equal(both[nb], new[nb])
    # nothing appended: nothing changes
    assert np.array_equal(oracle_mod.graph_append(emb[:n_old], old), old)
    # a store that starts empty: append equals build
    assert np.array_equal(oracle_mod.graph_append(emb[:50], np.zeros((0, deg), np.int32)), oracle_mod.knn_graph(emb[:50], deg))


# ------------------------------------------------------------------------------------------------ removed rows
def test_retrieval_with_removed_rows_is_retrieval_over_the_rows_that_remain(oracle_mod):
    """Masked retrieval reduces to the pinned plain routine on the compacted matrix with its row -> id map, and to a
    brute-force numpy ranking; removed rows never appear, ties still go to the lower id, short stores are padded."""
    rng = np.random.default_rng(8)
    for dtype, dim, n in (("float32", 64, 500), ("float16", 136, 300)):
        emb = synth.embeddings(8, n, dim, dtype)
        emb[200] = emb[17]
        emb[250] = emb[17]
        q = synth.queries(8, 3, dim, dtype)
        q[0] = emb[17]
        removed = rng.random(n) < 0.3
        removed[17] = True  # the best match of query 0 is gone: its copies move up, lower id first
        removed[[200, 250]] = False
        keep = np.flatnonzero(~removed)
        for k in (1, 7, len(keep), len(keep) + 5):
            ids, sc = oracle_mod.retrieve(emb, q, k, removed=removed)
            want_ids, want_sc = oracle_mod.retrieve(emb[keep], q, k, row_ids=keep.astype(np.int32))
            assert np.array_equal(ids, want_ids) and np.array_equal(sc, want_sc)
            assert not np.isin(ids[ids >= 0], np.flatnonzero(removed)).any()
        ids, _ = oracle_mod.retrieve(emb, q, 5, removed=removed)
        assert ids[0, :2].tolist() == [200, 250]
        s = emb.astype(np.float64) @ q[1].astype(np.float64)
        s[removed] = -np.inf
        order = np.lexsort((np.arange(n), -s))[:5]
        assert np.array_equal(oracle_mod.retrieve(emb, q[1:2], 5, removed=removed)[0][0], order)
    everything = np.ones(20, bool)
    ids, sc = oracle_mod.retrieve(emb[:20], q[:1], 3, removed=everything)
    assert ids.tolist() == [[-1, -1, -1]] and sc.tolist() == [[0.0, 0.0, 0.0]]


@pytest.mark.parametrize("exact", [False, True])
def test_search_walks_through_removed_rows_but_never_returns_them(oracle_mod, exact):
    # the path graph of the hand-followed walk: rows 64..66, on the way from the entry 61 to the target 70, are removed;
    # the walk still gets to 70 through them (same steps, same rows scored), and they are missing from the result
    n = 100
    emb = arc(n)
    path = np.array([[i - 1 if i > 0 else -1, i + 1 if i + 1 < n else -1] for i in range(n)], np.int32)
    q = emb[70:71].copy()
    removed = np.zeros(n, bool)
    removed[[64, 65, 66]] = True
    plain = oracle_mod.ann_search(emb, path, q, 4, beam=8, parents=1, n_entry=1, max_iters=50, exact=exact)
    gone = oracle_mod.ann_search(emb, path, q, 4, beam=8, parents=1, n_entry=1, max_iters=50, exact=exact, removed=removed)
    assert gone.iters[0] == plain.iters[0] and gone.scored[0] == plain.scored[0]
    assert gone.ids[0, 0] == 70 and not np.isin(gone.ids[0], [64, 65, 66]).any()
    # removing the target itself: the next best rows are returned
    removed[70] = True
    res = oracle_mod.ann_search(emb, path, q, 2, beam=8, parents=1, n_entry=1, max_iters=50, exact=exact, removed=removed)
    assert sorted(res.ids[0].tolist()) == [69, 71]
    # complete graph and a list as long as the store: the walk sees every row, so the result is the masked exact ranking
    m, dim, k = 120, 64, 9
    e2 = synth.embeddings(9, m, dim, "float32")
    complete = np.array([[c for c in range(m) if c != r] for r in range(m)], np.int32)
    q2 = synth.queries(9, 3, dim, "float32")
    rem2 = np.random.default_rng(9).random(m) < 0.25
    res = oracle_mod.ann_search(e2, complete, q2, k, beam=m, parents=4, n_entry=m, max_iters=3, exact=exact, removed=rem2)
    want, _ = oracle_mod.retrieve(e2, q2, k, removed=rem2)
    assert np.array_equal(res.ids, want)
    # a list shorter than the removed rows in front: fewer than k rows can be returned, the rest is padding
    rem3 = np.zeros(m, bool)
    best = oracle_mod.retrieve(e2, q2[:1], 6)[0][0]
    rem3[best[:5]] = True
    res = oracle_mod.ann_search(e2, complete, q2[:1], 4, beam=6, parents=4, n_entry=m, max_iters=3, exact=exact, removed=rem3)
    assert res.ids[0].tolist() == [int(best[5]), -1, -1, -1]


def test_recall_after_removing_a_tenth_of_the_rows(oracle_mod):
    n, dim, k = 3000, 64, 10
    emb = synth.embeddings_low_rank(10, n, dim, "float32", intrinsic_dim=8)
    g = oracle_mod.knn_graph(emb, 16)
    q = synth.queries_near_rows(10, emb, 20)
    removed = np.random.default_rng(10).random(n) < 0.1
    want, _ = oracle_mod.retrieve(emb, q, k, removed=removed)
    got = oracle_mod.ann_search(emb, g, q, k, beam=96, parents=2, n_entry=16, max_iters=200, removed=removed).ids
    assert not np.isin(got[got >= 0], np.flatnonzero(removed)).any()
    recall = np.mean([len(set(got[i]) & set(want[i])) / k for i in range(len(q))])
    assert recall > 0.9
    # a graph built after the removals lists no removed row; removed rows keep lists of their own
    g2 = oracle_mod.knn_graph(emb, 16, removed=removed)
    assert not np.isin(g2, np.flatnonzero(removed)).any() and np.all(g2[np.flatnonzero(removed)[0]] >= 0)
    keep = np.flatnonzero(~removed)
    sub = oracle_mod.knn_graph(emb[keep], 16)
    assert np.array_equal(g2[keep[5]], keep[sub[5]])  # an alive row's list = its list in the compacted store
