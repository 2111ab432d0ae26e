"""Pins for the oracle's attention and score arithmetic (Eq. 2, last row)."""
import math

import numpy as np
import torch

from oracle.st3_oracle import attend, visual_mass


def _rand(seed, H, T, D):
    r = np.random.default_rng(seed)
    return r.standard_normal((H, D)), r.standard_normal((H, T, D)), r.standard_normal((H, T, D))


def test_against_naive_long_double_without_max_subtraction():
    q, K, V = _rand(0, 3, 17, 8)
    out, p = attend(q, K, V)
    ql, Kl, Vl = q.astype(np.longdouble), K.astype(np.longdouble), V.astype(np.longdouble)
    for h in range(3):
        w = np.zeros(17, dtype=np.longdouble)
        for j in range(17):
            acc = np.longdouble(0)
            for d in range(8):
                acc += ql[h, d] * Kl[h, j, d]
            w[j] = np.exp(acc / np.sqrt(np.longdouble(8)))
        w = w / w.sum()
        ref = np.zeros(8, dtype=np.longdouble)
        for j in range(17):
            ref += w[j] * Vl[h, j]
        assert np.allclose(p[h], w.astype(np.float64), rtol=1e-12, atol=1e-15)
        assert np.allclose(out[h], ref.astype(np.float64), rtol=1e-12, atol=1e-14)


def test_against_torch_sdpa():
    q, K, V = _rand(1, 4, 33, 16)
    out, _ = attend(q, K, V)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[:, None, :], torch.from_numpy(K), torch.from_numpy(V))[:, 0, :]
    assert np.allclose(out, ref.numpy(), rtol=1e-11, atol=1e-13)


def test_causal_last_row_equals_decode_row():
    """The decode query is the last row of a causally masked square attention (Eq. 2)."""
    r = np.random.default_rng(2)
    T, D = 9, 4
    X = r.standard_normal((1, T, D))
    Kx, Vx = r.standard_normal((1, T, D)), r.standard_normal((1, T, D))
    full = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(X), torch.from_numpy(Kx), torch.from_numpy(Vx), is_causal=True)
    out, _ = attend(X[:, -1, :], Kx, Vx)
    assert np.allclose(out[0], full[0, -1].numpy(), rtol=1e-11, atol=1e-13)


def test_single_key_returns_its_value_and_equal_keys_average():
    q, K, V = _rand(3, 2, 1, 8)
    out, p = attend(q, K, V)
    assert np.array_equal(p, np.ones((2, 1)))
    assert np.allclose(out, V[:, 0, :], rtol=0, atol=0)
    q, K, V = _rand(4, 2, 6, 8)
    K[:] = K[:, :1, :]
    out, p = attend(q, K, V)
    assert np.allclose(p, 1.0 / 6.0, rtol=1e-14)
    assert np.allclose(out, V.mean(axis=1), rtol=1e-13)


def test_shift_invariance_and_large_logits_do_not_overflow():
    q, K, V = _rand(5, 2, 12, 8)
    out0, _ = attend(q, K, V)
    out1, p1 = attend(200.0 * q, K, V)           # logits of order 1e3: exp() would overflow unshifted
    assert np.all(np.isfinite(out1)) and np.allclose(p1.sum(axis=1), 1.0)
    # adding a constant vector c to every key shifts every logit of a head equally: no change
    c = np.random.default_rng(6).standard_normal((2, 1, 8))
    out2, _ = attend(q, K + c, V)
    assert np.allclose(out0, out2, rtol=1e-10, atol=1e-12)


def test_mass_accounts_for_all_probability():
    H, T, D, sys_len, nv = 5, 40, 8, 7, 21
    q, K, V = _rand(7, H, T, D)
    _, p = attend(q, K, V)
    m = visual_mass(p, sys_len, nv)
    assert m.shape == (nv,) and np.all(m >= 0) and np.all(m <= H)
    non_visual = p[:, :sys_len].sum() + p[:, sys_len + nv:].sum()
    assert abs(m.sum() + non_visual - H) < 1e-12
    # transposed-operand guard: mass is a per-token sum over heads, not per-head sum over tokens
    assert np.allclose(m, np.array([sum(p[h, sys_len + i] for h in range(H)) for i in range(nv)]))


def test_inherited_attention_is_the_sources_probabilities_on_own_values():
    from oracle.st3_oracle import attend_inherited
    r = np.random.default_rng(31)
    H, T, D = 3, 14, 8
    qs, Ks, Vs = r.standard_normal((H, D)), r.standard_normal((H, T, D)), r.standard_normal((H, T, D))
    Vl = r.standard_normal((H, T, D))
    _, p = attend(qs, Ks, Vs)
    want = np.stack([sum(p[h, j] * Vl[h, j] for j in range(T)) for h in range(H)])
    assert np.allclose(attend_inherited(qs, Ks, Vl), want, rtol=1e-13, atol=1e-15)
    # with its own query, keys and values a layer "inherits" plain attention
    assert np.allclose(attend_inherited(qs, Ks, Vs), attend(qs, Ks, Vs)[0], rtol=1e-13, atol=1e-15)
    # library special case: SDPA with the source's q, k and the lazy layer's v
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qs)[:, None, :], torch.from_numpy(Ks), torch.from_numpy(Vl))[:, 0, :]
    assert np.allclose(attend_inherited(qs, Ks, Vl), ref.numpy(), rtol=1e-11, atol=1e-13)


def test_causal_attention_against_sdpa_and_its_last_row_against_attend():
    from oracle.st3_oracle import causal_attention
    r = np.random.default_rng(41)
    H, T, D = 2, 19, 8
    Q, K, V = r.standard_normal((H, T, D)), r.standard_normal((H, T, D)), r.standard_normal((H, T, D))
    out, A = causal_attention(Q, K, V)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(Q), torch.from_numpy(K),
                                                           torch.from_numpy(V), is_causal=True)
    assert np.allclose(out, ref.numpy(), rtol=1e-11, atol=1e-13)
    assert np.allclose(A.sum(axis=2), 1.0) and np.all(np.triu(A, k=1) == 0)      # rows sum to 1, no look-ahead
    assert np.allclose(out[:, 0], V[:, 0])                                       # the first token sees itself only
    o_last, p_last = attend(Q[:, -1], K, V)                                      # the decode row of Eq. 2
    assert np.allclose(out[:, -1], o_last, rtol=1e-12, atol=1e-14) and np.allclose(A[:, -1], p_last, rtol=1e-12)
    # brute force of one entry
    i, h = 7, 1
    w = np.array([math.exp(float(Q[h, i] @ K[h, j]) / math.sqrt(D)) for j in range(i + 1)])
    assert np.allclose(out[h, i], (w[:, None] * V[h, :i + 1]).sum(axis=0) / w.sum(), rtol=1e-12)
