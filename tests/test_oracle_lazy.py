"""Pins for the oracle's decode step of a lazy layer (QK heredity: Eq. 6, Algorithm 2).

The expected values are written out from the definition with explicit loops: the probabilities
come from the SOURCE layer's query and keys (the source's newly appended key included), they are
applied to the lazy layer's OWN values (its newly appended value included), and the eviction that
the stage's pruning layer decided happens after the layer has attended.
"""
import math

import numpy as np
import pytest

from oracle import st3_oracle as O


def _cache(r, H, D, n_sys, ids, n_txt):
    n = len(ids)
    mk = lambda t: r.standard_normal((H, t, D))
    return O.LayerCache(K_sys=mk(n_sys), V_sys=mk(n_sys), K_vis=mk(n), V_vis=mk(n), ids=np.array(ids, dtype=np.int64),
                        K_txt=mk(n_txt), V_txt=mk(n_txt))


def _copy(c):
    return O.LayerCache(**{k: np.array(getattr(c, k), copy=True) for k in
                           ("K_sys", "V_sys", "K_vis", "V_vis", "ids", "K_txt", "V_txt")})


def _explicit(q_src, K_src_rows, V_own_rows):
    """sum_j p[h, j] V_own[h, j] with p = softmax_j(q_src[h] . K_src[h, j] / sqrt(D)), loop by loop."""
    H, T, D = K_src_rows.shape
    out = np.zeros((H, D))
    for h in range(H):
        w = [math.exp(sum(q_src[h, d] * K_src_rows[h, j, d] for d in range(D)) / math.sqrt(D)) for j in range(T)]
        z = sum(w)
        for j in range(T):
            out[h] += (w[j] / z) * V_own_rows[h, j]
    return out


def _exhaustive_top(scores, ids, k):
    """i is kept  <=>  fewer than k rows beat it (higher score, or equal score and lower original index)."""
    n = len(scores)
    return [i for i in range(n)
            if sum(1 for j in range(n) if scores[j] > scores[i] or (scores[j] == scores[i] and ids[j] < ids[i])) < k]


def _setup(seed=0, H=2, D=4, n_sys=2, ids=(7, 2, 9, 4, 11, 0), n_txt=3):
    r = np.random.default_rng(seed)
    lazy = _cache(r, H, D, n_sys, ids, n_txt)
    src = _cache(r, H, D, n_sys, ids, n_txt)
    q_src, k_src_new, v_new = r.standard_normal((H, D)), r.standard_normal((H, D)), r.standard_normal((H, D))
    # the source layer has appended its own new key for this step (its value plays no part here)
    src.K_txt = np.concatenate([src.K_txt, k_src_new[:, None, :]], axis=1)
    src.V_txt = np.concatenate([src.V_txt, np.full((H, 1, D), np.nan)], axis=1)
    return lazy, src, q_src, v_new


def test_output_is_the_sources_probabilities_on_own_values_with_both_new_rows():
    lazy, src, q_src, v_new = _setup()
    before = _copy(lazy)
    out = O.decode_step_lazy(lazy, src, q_src, v_new, n_target=6, select_scores=np.zeros(6))
    K_rows = np.concatenate([src.K_sys, src.K_vis, src.K_txt], axis=1)                       # new key is the last row
    V_rows = np.concatenate([before.V_sys, before.V_vis, before.V_txt, v_new[:, None, :]], axis=1)
    assert np.allclose(out, _explicit(q_src, K_rows, V_rows), rtol=1e-12, atol=1e-14)
    # the new value went to the end of the text region and nothing else moved
    assert lazy.V_txt.shape[1] == before.V_txt.shape[1] + 1 and np.array_equal(lazy.V_txt[:, -1], v_new)
    assert np.array_equal(lazy.V_txt[:, :-1], before.V_txt) and np.array_equal(lazy.V_sys, before.V_sys)
    assert np.array_equal(lazy.V_vis, before.V_vis) and np.array_equal(lazy.ids, before.ids)
    # wrong-operand guards: neither the source's values nor the lazy layer's own keys give this result
    wrong_v = np.concatenate([src.V_sys, src.V_vis, src.V_txt[:, :-1], v_new[:, None, :]], axis=1)
    assert not np.allclose(out, _explicit(q_src, K_rows, wrong_v), rtol=1e-3)
    own_k = np.concatenate([before.K_sys, before.K_vis, before.K_txt, src.K_txt[:, -1:]], axis=1)
    assert not np.allclose(out, _explicit(q_src, own_k, V_rows), rtol=1e-3)
    # dropping the source's new key or the lazy layer's new value changes the result
    assert not np.allclose(out, _explicit(q_src, K_rows[:, :-1], V_rows[:, :-1]), rtol=1e-3)


def test_the_lazy_layers_own_keys_are_never_read():
    lazy, src, q_src, v_new = _setup(seed=1)
    ref = O.decode_step_lazy(_copy(lazy), src, q_src, v_new, 4, np.arange(6.0))
    lazy.K_sys[:] = np.nan
    lazy.K_vis[:] = np.nan
    lazy.K_txt[:] = np.nan
    out = O.decode_step_lazy(lazy, src, q_src, v_new, 4, np.arange(6.0))
    assert np.all(np.isfinite(out)) and np.array_equal(out, ref)


def test_eviction_comes_after_attending_and_follows_the_given_scores():
    lazy, src, q_src, v_new = _setup(seed=2)
    ids = lazy.ids.copy()
    # row 3 is about to be evicted (lowest score) but carries almost all of the probability: the output must
    # still contain its value, i.e. the layer attends over the rows held BEFORE the eviction
    src.K_vis[:, 3] = 6.0 * q_src
    lazy.V_vis[:, 3] = 100.0
    scores = np.array([0.5, 0.9, 0.5, 0.1, 0.5, 0.7])            # three-way tie at 0.5: ids 7, 9, 11
    before = _copy(lazy)
    out = O.decode_step_lazy(lazy, src, q_src, v_new, n_target=3, select_scores=scores)
    assert np.all(out > 50.0)
    K_rows = np.concatenate([src.K_sys, src.K_vis, src.K_txt], axis=1)
    V_rows = np.concatenate([before.V_sys, before.V_vis, before.V_txt, v_new[:, None, :]], axis=1)
    assert np.allclose(out, _explicit(q_src, K_rows, V_rows), rtol=1e-12, atol=1e-12)
    kept = _exhaustive_top(scores, ids, 3)                       # positions 1 (0.9), 5 (0.7) and, of the tie, id 7
    assert kept == [0, 1, 5]
    assert lazy.ids.tolist() == [int(ids[i]) for i in kept]
    assert np.array_equal(lazy.V_vis, before.V_vis[:, kept]) and np.array_equal(lazy.K_vis, before.K_vis[:, kept])
    assert lazy.n_cur == 3


@pytest.mark.parametrize("n_target", [0, 6, 9])
def test_target_counts_at_the_ends(n_target):
    lazy, src, q_src, v_new = _setup(seed=3)
    before = _copy(lazy)
    O.decode_step_lazy(lazy, src, q_src, v_new, n_target, np.arange(6.0))
    want = min(6, n_target)
    assert lazy.n_cur == want
    if want == 6:
        assert np.array_equal(lazy.ids, before.ids) and np.array_equal(lazy.V_vis, before.V_vis)


def test_exhaustive_selection_on_random_scores_with_ties():
    r = np.random.default_rng(4)
    for trial in range(20):
        n = int(r.integers(1, 12))
        ids = r.permutation(40)[:n]
        lazy, src, q_src, v_new = _setup(seed=10 + trial, ids=tuple(int(i) for i in ids))
        scores = r.integers(0, 4, size=n).astype(np.float64)      # many equal scores
        k = int(r.integers(0, n + 1))
        O.decode_step_lazy(lazy, src, q_src, v_new, k, scores)
        assert lazy.ids.tolist() == [int(ids[i]) for i in _exhaustive_top(scores, ids, k)]


def test_rows_of_source_and_lazy_layer_must_name_the_same_tokens():
    lazy, src, q_src, v_new = _setup(seed=5)
    src.ids = src.ids[::-1].copy()
    with pytest.raises(AssertionError):
        O.decode_step_lazy(lazy, src, q_src, v_new, 6, np.zeros(6))


def test_a_layer_that_inherits_from_itself_is_the_plain_decode_step():
    """Special case: with source = the layer itself (same q, keys) the lazy step reduces to decode_step."""
    r = np.random.default_rng(6)
    H, D = 2, 4
    c = _cache(r, H, D, 2, (3, 1, 8, 5), 2)
    q, kn, vn = r.standard_normal((H, D)), r.standard_normal((H, D)), r.standard_normal((H, D))
    plain = _copy(c)
    out_plain, mass, _ = O.decode_step(plain, q, kn, vn, 2)
    src = _copy(c)
    src.K_txt = np.concatenate([src.K_txt, kn[:, None, :]], axis=1)
    src.V_txt = np.concatenate([src.V_txt, np.zeros((H, 1, D))], axis=1)
    out_lazy = O.decode_step_lazy(c, src, q, vn, 2, mass)
    assert np.allclose(out_lazy, out_plain, rtol=1e-13, atol=1e-15)
    assert np.array_equal(c.ids, plain.ids) and np.array_equal(c.V_vis, plain.V_vis)
