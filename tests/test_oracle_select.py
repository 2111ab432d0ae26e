"""Pins for Top(G, alpha) (Eq. 3) with the lower-index tie-break, and for cache bookkeeping."""
import numpy as np
import pytest

from oracle import st3_oracle as O
from oracle.st3_oracle import select_top, boundary_scores, prefill_select, decode_step


def _exhaustive(scores, ids, k):
    """i is kept iff fewer than k tokens beat it (higher score, or equal score and lower id)."""
    n = len(scores)
    keep = []
    for i in range(n):
        beat = sum(1 for j in range(n)
                   if scores[j] > scores[i] or (scores[j] == scores[i] and ids[j] < ids[i]))
        if beat < k:
            keep.append(i)
    return np.array(keep, dtype=np.int64)


@pytest.mark.parametrize("seed", range(6))
def test_matches_exhaustive_definition_with_ties(seed):
    r = np.random.default_rng(seed)
    n = int(r.integers(1, 40))
    scores = r.integers(0, 5, size=n).astype(np.float64) / 4.0     # many exact ties
    ids = r.permutation(100)[:n]
    for k in range(0, n + 1):
        assert np.array_equal(select_top(scores, ids, k), _exhaustive(scores, ids, k))


def test_all_equal_keeps_lowest_ids_and_extremes():
    ids = np.array([9, 2, 7, 4, 0, 5])
    s = np.full(6, 0.25)
    kept = select_top(s, ids, 3)
    assert sorted(ids[kept].tolist()) == [0, 2, 4]
    assert len(select_top(s, ids, 0)) == 0
    assert np.array_equal(select_top(s, ids, 6), np.arange(6))
    assert np.array_equal(select_top(s, ids, 99), np.arange(6))


def test_no_ties_equals_sort():
    r = np.random.default_rng(11)
    s = r.random(50)
    kept = select_top(s, np.arange(50), 20)
    assert set(kept.tolist()) == set(np.argsort(-s)[:20].tolist())
    sk, sk1 = boundary_scores(s, np.arange(50), 20)
    srt = np.sort(s)[::-1]
    assert sk == srt[19] and sk1 == srt[20]


def test_prefill_and_decode_bookkeeping():
    r = np.random.default_rng(12)
    H, D, sys_len, nv, text = 2, 4, 3, 10, 4
    T0 = sys_len + nv + text
    K, V = r.standard_normal((H, T0, D)), r.standard_normal((H, T0, D))
    q = r.standard_normal((H, D))
    out, mass, c = prefill_select(q, K, V, sys_len, nv, 6)
    assert c.n_cur == 6 and mass.shape == (nv,)
    # kept rows are bit-identical to the source rows their ids name
    assert np.array_equal(c.K_vis, K[:, sys_len + c.ids]) and np.array_equal(c.V_vis, V[:, sys_len + c.ids])
    assert np.array_equal(c.K_sys, K[:, :sys_len]) and np.array_equal(c.K_txt, K[:, sys_len + nv:])
    assert set(c.ids.tolist()) == set(np.argsort(-mass)[:6].tolist())
    kn, vn = r.standard_normal((H, D)), r.standard_normal((H, D))
    ids0 = c.ids.copy()
    out1, m1, before = decode_step(c, r.standard_normal((H, D)), kn, vn, 4)
    assert np.array_equal(before, ids0) and m1.shape == (6,)
    assert c.n_cur == 4 and set(c.ids.tolist()) <= set(ids0.tolist())
    assert c.K_txt.shape[1] == text + 1 and np.array_equal(c.K_txt[:, -1], kn)
    assert np.array_equal(c.K_vis, K[:, sys_len + c.ids])
    # a target above the current count never grows the cache
    decode_step(c, r.standard_normal((H, D)), kn, vn, 9)
    assert c.n_cur == 4
    # empty visual span is legal (beta = 0)
    decode_step(c, r.standard_normal((H, D)), kn, vn, 0)
    assert c.n_cur == 0
    o, m, _ = decode_step(c, r.standard_normal((H, D)), kn, vn, 0)
    assert m.shape == (0,) and np.all(np.isfinite(o))


def test_rank_order_prefixes_are_the_top_sets():
    from oracle.st3_oracle import rank_order
    r = np.random.default_rng(21)
    scores = r.integers(0, 6, size=30).astype(np.float64)         # ties
    ids = r.permutation(64)[:30]
    order = rank_order(scores, ids)
    assert sorted(order.tolist()) == list(range(30))
    for a, b in zip(order[:-1], order[1:]):                       # sorted by (score desc, id asc)
        assert scores[a] > scores[b] or (scores[a] == scores[b] and ids[a] < ids[b])
    for k in range(31):
        assert set(order[:k].tolist()) == set(_exhaustive(scores, ids, k).tolist())


def test_static_rank_decode_truncates_the_saved_order():
    from oracle.st3_oracle import decode_step_static, attend
    r = np.random.default_rng(22)
    H, D, sys_len, nv, text = 2, 4, 2, 12, 3
    T0 = sys_len + nv + text
    K, V = r.standard_normal((H, T0, D)), r.standard_normal((H, T0, D))
    out, mass, c = prefill_select(r.standard_normal((H, D)), K, V, sys_len, nv, 8, rank_ordered=True)
    assert np.all(np.diff(mass[c.ids]) <= 0)                      # best first
    assert np.array_equal(c.K_vis, K[:, sys_len + c.ids])
    ids0 = c.ids.copy()
    q, kn, vn = r.standard_normal((H, D)), r.standard_normal((H, D)), r.standard_normal((H, D))
    o = decode_step_static(c, q, kn, vn, 5)
    assert np.array_equal(c.ids, ids0[:5])                        # a prefix, nothing re-scored
    # it attended over exactly [S | first 5 of the order | I | new token]
    rows = list(range(sys_len)) + (sys_len + ids0[:5]).tolist() + list(range(sys_len + nv, T0))
    Kx = np.concatenate([K[:, rows], kn[:, None]], axis=1)
    Vx = np.concatenate([V[:, rows], vn[:, None]], axis=1)
    assert np.allclose(o, attend(q, Kx, Vx)[0], rtol=1e-13, atol=1e-15)
    decode_step_static(c, q, kn, vn, 9)                           # never grows
    assert c.n_cur == 5


def test_externally_scored_prefill_prunes_before_it_attends():
    from oracle.st3_oracle import prefill_select_scored, attend
    r = np.random.default_rng(23)
    H, D, sys_len, nv, text = 2, 4, 2, 11, 3
    T0 = sys_len + nv + text
    K, V = r.standard_normal((H, T0, D)), r.standard_normal((H, T0, D))
    q = r.standard_normal((H, D))
    scores = r.permutation(nv).astype(np.float64)                  # distinct: top-5 = the 5 largest
    out, c = prefill_select_scored(q, K, V, sys_len, nv, 5, scores)
    want = np.sort(np.argsort(-scores)[:5])
    assert np.array_equal(c.ids, want)
    rows = list(range(sys_len)) + (sys_len + want).tolist() + list(range(sys_len + nv, T0))
    assert np.allclose(out, attend(q, K[:, rows], V[:, rows])[0], rtol=1e-13, atol=1e-15)
    # keeping everything reduces to plain attention over the whole prompt
    out_all, c_all = prefill_select_scored(q, K, V, sys_len, nv, nv, scores)
    assert np.allclose(out_all, attend(q, K, V)[0], rtol=1e-13, atol=1e-15) and c_all.n_cur == nv
    # fed with the layer's own scores it keeps what prefill_select keeps
    o_self, m_self, c_self = prefill_select(q, K, V, sys_len, nv, 5)
    _, c_fed = prefill_select_scored(q, K, V, sys_len, nv, 5, m_self)
    assert np.array_equal(c_fed.ids, c_self.ids)
    _, c_rank = prefill_select_scored(q, K, V, sys_len, nv, 5, scores, rank_ordered=True)
    assert c_rank.ids.tolist() == np.argsort(-scores)[:5].tolist()


def test_follower_layers_adopt_the_pruning_layers_choice():
    """select_scores: a layer between two pruning layers keeps what the pruning layer's scores keep."""
    r = np.random.default_rng(24)
    H, D, sys_len, nv, text = 2, 4, 1, 9, 2
    T0 = sys_len + nv + text
    mk = lambda: (r.standard_normal((H, D)), r.standard_normal((H, T0, D)), r.standard_normal((H, T0, D)))
    qa, Ka, Va = mk()
    qb, Kb, Vb = mk()
    oa, ma, ca = prefill_select(qa, Ka, Va, sys_len, nv, 5)
    ob, mb, cb = prefill_select(qb, Kb, Vb, sys_len, nv, 5, select_scores=ma)
    assert np.array_equal(ca.ids, cb.ids)                                  # same tokens ...
    assert np.array_equal(cb.K_vis, Kb[:, sys_len + cb.ids])               # ... of the follower's own rows
    ob_own, mb_own, _ = prefill_select(qb, Kb, Vb, sys_len, nv, 5)
    assert np.array_equal(ob, ob_own) and np.array_equal(mb, mb_own)       # attention itself is unchanged
    kn, vn = r.standard_normal((H, D)), r.standard_normal((H, D))
    _, m1, _ = decode_step(ca, r.standard_normal((H, D)), kn, vn, 3)
    decode_step(cb, r.standard_normal((H, D)), kn, vn, 3, select_scores=m1)
    assert np.array_equal(ca.ids, cb.ids)


def test_overlap_n_closed_forms_and_brute_force():
    """Eq. 10 on sets with known intersections, and against a brute-force count on top-K sets of random scores."""
    assert O.overlap_n([1, 2, 3, 4], [1, 2, 3, 4]) == 1.0
    assert O.overlap_n([1, 2, 3, 4], [5, 6, 7, 8]) == 0.0
    assert O.overlap_n([1, 2, 3, 4], [3, 4, 5, 6]) == 0.5
    assert O.overlap_n([7, 8, 9], [9]) == pytest.approx(1 / 3)          # the denominator is the first step's set
    rng = np.random.default_rng(3)
    ids = np.arange(200)
    for k in (1, 17, 100, 200):
        s1, sn = rng.normal(size=200), rng.normal(size=200)
        t1, tn = ids[O.select_top(s1, ids, k)], ids[O.select_top(sn, ids, k)]
        brute = sum(1 for i in np.argsort(-s1, kind="stable")[:k] if i in set(np.argsort(-sn, kind="stable")[:k].tolist())) / k
        assert O.overlap_n(t1, tn) == pytest.approx(brute)
    # the same scores at both steps: the top-K does not move
    s = rng.normal(size=200)
    assert O.overlap_n(ids[O.select_top(s, ids, 50)], ids[O.select_top(s, ids, 50)]) == 1.0
