"""Shared test helpers: oracle runners over synthetic workloads and the kept-set acceptance rule."""
from __future__ import annotations

import numpy as np
import torch

from oracle import st3_oracle as O
from synth import SynthInputs, Workload


def make_schedule(wl: Workload, **kw) -> O.Schedule:
    args = dict(num_layers=wl.num_layers, num_visual=wl.num_visual, stride=wl.stride,
                step_ratio_bp=wl.step_ratio_bp, tau=wl.tau, first_ratio_bp=wl.first_ratio_bp,
                first_prune_layer=wl.first_prune_layer)
    args.update(kw)
    return O.Schedule(**args)


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_prefill_unit(wl: Workload, g: SynthInputs, sched: O.Schedule, b: int, l: int):
    """Prefill-select of one (sequence, layer) on regenerated inputs."""
    t0 = wl.sys_len + wl.num_visual + int(g.text_len[b])
    K, V = g.kv_rows([b], [l], range(t0))
    q = g.queries([0], [l])[0, 0, b]
    return O.prefill_select(f64(q), f64(K[0, 0]), f64(V[0, 0]), wl.sys_len, wl.num_visual, sched.n0(l))


def oracle_decode_unit(wl: Workload, g: SynthInputs, sched: O.Schedule, cache: O.LayerCache,
                       b: int, l: int, step: int):
    q = g.queries([step], [l])[0, 0, b]
    kn, vn = g.new_kv([step], [l])
    return O.decode_step(cache, f64(q), f64(kn[0, 0, b]), f64(vn[0, 0, b]), sched.n(l, step))


def rebuild_cache(wl: Workload, g: SynthInputs, b: int, l: int, ids, steps_done: int) -> O.LayerCache:
    """Oracle cache of (b, l) after `steps_done` decode steps, given the kept visual ids."""
    text = int(g.text_len[b])
    ids = np.asarray(ids, dtype=np.int64)
    toks_txt = list(range(wl.sys_len + wl.num_visual, wl.sys_len + wl.num_visual + text)) + \
        [g.gen_token(s) for s in range(1, steps_done + 1)]
    Ks, Vs = g.kv_rows([b], [l], range(wl.sys_len))
    Kv, Vv = g.kv_rows([b], [l], (wl.sys_len + ids).tolist())
    Kt, Vt = g.kv_rows([b], [l], toks_txt)
    return O.LayerCache(K_sys=f64(Ks[0, 0]), V_sys=f64(Vs[0, 0]), K_vis=f64(Kv[0, 0]), V_vis=f64(Vv[0, 0]),
                        ids=ids.copy(), K_txt=f64(Kt[0, 0]), V_txt=f64(Vt[0, 0]))


def check_kept(mass: np.ndarray, ids_before: np.ndarray, k: int, got_ids, rel: float = 1e-3):
    """Acceptance rule for a selection.

    With s_k, s_{k+1} the oracle's scores on either side of the cut: if their gap exceeds
    rel*|s_k| the kept set must equal the oracle's exactly; otherwise the position is a
    near-tie and the two sets may differ only inside the band |s_i - s_k| <= rel*|s_k|.
    Returns "exact" or "near-tie"; raises AssertionError otherwise.
    """
    got = set(int(i) for i in got_ids)
    n = len(mass)
    k = min(k, n)
    assert len(got) == k, f"kept {len(got)} rows, schedule says {k}"
    assert got <= set(int(i) for i in ids_before), "kept an id that was not in the cache"
    want_pos = O.select_top(mass, ids_before, k)
    want = set(int(i) for i in ids_before[want_pos])
    if got == want:
        return "exact"
    s_k, s_k1 = O.boundary_scores(mass, ids_before, k)
    assert s_k is not None and s_k1 is not None
    assert (s_k - s_k1) <= rel * abs(s_k), \
        f"kept set differs with a clear gap: s_k={s_k} s_k+1={s_k1} diff={sorted(got ^ want)}"
    by_id = {int(i): float(m) for i, m in zip(ids_before, mass)}
    for i in got ^ want:
        assert abs(by_id[i] - s_k) <= rel * abs(s_k), f"id {i} differs outside the near-tie band"
    return "near-tie"
