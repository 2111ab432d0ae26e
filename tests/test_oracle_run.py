"""Run-long invariants of the oracle on the tiny workload, and synthetic-input determinism."""
import numpy as np
import pytest
import torch

from oracle import st3_oracle as O
from synth import SynthInputs, get_workload
from helpers import make_schedule, oracle_prefill_unit, oracle_decode_unit, rebuild_cache, f64, check_kept


@pytest.mark.parametrize("tau", [50.0, 10.0])
def test_tiny_run_invariants(tau):
    wl = get_workload("tiny").scaled(tau=tau)
    g = SynthInputs(wl)
    sched = make_schedule(wl)
    out, mass, c = oracle_prefill_unit(wl, g, sched, 0, 0)
    assert c.n_cur == 288 == sched.n0(0)
    sys_sum = c.K_sys.sum()
    prev = set(c.ids.tolist())
    planted = set(g.planted(0, 0).tolist())
    assert planted <= prev                       # sanity: +2 logit tokens survive a 50% cut
    for t in range(1, wl.decode_steps + 1):
        out, mass, before = oracle_decode_unit(wl, g, sched, c, 0, 0, t)
        assert np.all(np.isfinite(out))
        assert c.n_cur == sched.n(0, t)                            # count follows the schedule
        cur = set(c.ids.tolist())
        assert cur <= prev and len(cur) == len(c.ids)              # nested, unique
        assert all(0 <= i < wl.num_visual for i in cur)
        assert c.K_txt.shape[1] == int(g.text_len[0]) + t          # text / generated rows never pruned
        assert c.K_sys.sum() == sys_sum
        prev = cur
    if tau == 10.0:
        assert c.n_cur == 0                                        # beta = 0 once |O| >= tau


def test_teacher_forced_rebuild_equals_free_running_state():
    wl = get_workload("tiny")
    g = SynthInputs(wl)
    sched = make_schedule(wl)
    _, _, c = oracle_prefill_unit(wl, g, sched, 0, 0)
    for t in range(1, 4):
        oracle_decode_unit(wl, g, sched, c, 0, 0, t)
    r = rebuild_cache(wl, g, 0, 0, c.ids, 3)
    assert np.array_equal(r.K_vis, c.K_vis) and np.array_equal(r.V_txt, c.V_txt) and np.array_equal(r.K_sys, c.K_sys)
    o1, m1, _ = oracle_decode_unit(wl, g, sched, c, 0, 0, 4)
    o2, m2, _ = oracle_decode_unit(wl, g, sched, r, 0, 0, 4)
    assert np.array_equal(o1, o2) and np.array_equal(m1, m2) and np.array_equal(c.ids, r.ids)


def test_acceptance_rule():
    mass = np.array([0.5, 0.4, 0.3000001, 0.3, 0.1])
    ids = np.arange(5)
    assert check_kept(mass, ids, 2, [0, 1]) == "exact"
    assert check_kept(mass, ids, 3, [0, 1, 3]) == "near-tie"
    with pytest.raises(AssertionError):
        check_kept(mass, ids, 2, [0, 2])
    with pytest.raises(AssertionError):
        check_kept(mass, ids, 3, [0, 1])


def test_synth_is_a_pure_function_of_its_indices():
    wl = get_workload("llava15_7b")
    g1, g2 = SynthInputs(wl), SynthInputs(wl)
    K, V = g1.kv_rows([0], [5], range(wl.t0_max))
    Kb, Vb = g2.kv_rows([0], [4, 5], [40, 41, 600])
    assert torch.equal(K[0, 0][:, [40, 41, 600]], Kb[0, 1]) and torch.equal(V[0, 0][:, [40, 41, 600]], Vb[0, 1])
    Kp, Vp = g1.prompt_kv([5])
    assert torch.equal(Kp[0, 0], K[0, 0])
    q = g1.queries([0, 3], [5, 6])
    assert torch.equal(q[1, 0], g2.queries([3], [5])[0, 0])
    kn, vn = g1.new_kv([2], [5])
    kk, vv = g2.kv_rows([0], [5], [g2.gen_token(2)])
    assert torch.equal(kn[0, 0, 0], kk[0, 0, :, 0]) and torch.equal(vn[0, 0, 0], vv[0, 0, :, 0])
    # statistics: z ~ N(0,1); planted keys shifted by 2 along the query-mean direction
    z = f64(V[0, 0])
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    pl = g1.planted(0, 5)
    assert len(pl) == 28 and len(set(pl.tolist())) == 28
    qv = f64(g1.queries([1], [5])[0, 0, 0])
    logit = np.einsum("htd,hd->ht", f64(K[0, 0]), qv) / np.sqrt(wl.head_dim)
    vis = logit[:, wl.sys_len:wl.sys_len + wl.num_visual]
    rest = np.delete(vis, pl, axis=1)
    assert 1.6 < vis[:, pl].mean() - rest.mean() < 2.4


def test_text_lengths_and_patch_planting():
    g = SynthInputs(get_workload("llava15_7b_b32"))
    assert g.text_len.min() >= 16 and g.text_len.max() <= 128 and len(set(g.text_len.tolist())) > 8
    wl = get_workload("llava_next_b8")
    g = SynthInputs(wl)
    pl = g.planted(0, 0)
    assert len(pl) == 86 and pl.max() < 2880
    r, c = (pl % 576) // 24, pl % 24
    # clustered: almost every planted token has a planted 4-neighbour in the same tile
    s = set(pl.tolist())
    nb = sum(1 for i in pl if any((i + d) in s for d in (-1, 1, -24, 24)))
    assert nb >= 80
