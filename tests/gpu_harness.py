"""Drives the CUDA path through the C ABI on a synthetic workload and checks it against the oracle.

Parity is teacher-forced: before judging a step the oracle's cache for a (sequence, layer) unit is
rebuilt from the kept ids the GPU holds, so every step is compared on identical state; the kept
set after the step is judged with the near-tie acceptance rule.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import st3_oracle as O
from paper_2412_20105_b200 import binding as B
from synth import SynthInputs, Workload
from helpers import make_schedule, rebuild_cache, check_kept, f64

OUT_ABS_F32 = 2e-3          # max-abs bound for fp32 outputs
OUT_REL_BF16 = 2e-2         # relative bound for bf16 outputs ...
OUT_FLOOR_BF16 = 1e-2       # ... relative to max(|ref|, this floor)
MASS_RTOL, MASS_ATOL = 5e-4, 1e-9


def assert_out_close(got: np.ndarray, ref: np.ndarray, dtype: str, where=""):
    assert np.all(np.isfinite(got)), where
    if dtype == "f32":
        err = np.abs(got - ref).max()
        assert err <= OUT_ABS_F32, f"{where}: max-abs {err}"
    else:
        rel = np.abs(got - ref) / np.maximum(np.abs(ref), OUT_FLOOR_BF16)
        assert rel.max() <= OUT_REL_BF16, f"{where}: max-rel {rel.max()}"


def assert_rank_ordered(ref_mass, got_ids, where="", rel=1e-3):
    """The stored order is best-first by the oracle's scores; neighbours may swap only inside a near-tie."""
    m = np.asarray(ref_mass)[np.asarray(got_ids, dtype=np.int64)]
    for r in range(len(m) - 1):
        if m[r] > m[r + 1]:
            continue
        if m[r] == m[r + 1]:
            assert got_ids[r] < got_ids[r + 1], f"{where}: equal scores must be ordered by lower index (rank {r})"
        else:
            assert m[r + 1] - m[r] <= rel * abs(m[r + 1]), f"{where}: rank {r} out of order: {m[r]} < {m[r + 1]}"


class GpuRun:
    def __init__(self, wl: Workload, device="cuda:0", sched_kw=None, overlap=False, **cfg_overrides):
        """`overlap`: back-to-back steps overlap on the GPU (st3_set_overlap); the inputs of a step are then
        generated and synchronised before the step is enqueued, as that mode requires."""
        self.wl, self.dev = wl, torch.device(device)
        self.g = SynthInputs(wl)
        self.sched = make_schedule(wl, disable_trim=bool(cfg_overrides.get("disable_trim", 0)), **(sched_kw or {}))
        self.cfg = B.config_from_workload(wl, **cfg_overrides)
        self.ctx = B.Context(self.cfg, device)
        self.overlap = bool(overlap)
        self._ahead = {}
        B.st3_set_overlap(self.ctx.handle, self.overlap)
        self.L = wl.num_layers
        self.out = torch.empty(self.ctx.io_shape(), dtype=self.ctx.dtype, device=self.dev)
        self.stats = {"exact": 0, "near-tie": 0, "units": 0}
        self.static = bool(cfg_overrides.get("static_rank", 0))
        self.shared = bool(cfg_overrides.get("stage_shared", 0))
        self._src_mass = {}          # (b, layer, step) -> oracle scores of a pruning layer
        self.lazy_mask = int(cfg_overrides.get("lazy_mask", 0))

    def close(self):
        self.ctx.close()

    # ------------------------------------------------------------------ running
    def prefill(self, layers_per_call=None):
        wl, g = self.wl, self.g
        step = layers_per_call or self.L
        q0 = g.queries([0], device=self.dev)[0]
        for l0 in range(0, self.L, step):
            ls = list(range(l0, min(self.L, l0 + step)))
            K, V = g.prompt_kv(ls, device=self.dev)
            self.ctx.prefill_select(q0[l0:l0 + len(ls)].contiguous(), K, V, g.text_len.tolist(),
                                    self.out[l0:l0 + len(ls)], layer_begin=l0)
            del K, V
        self.q_cur = q0
        return self.out

    def prefill_scored(self, scores):
        """Prefill with caller-supplied scores [L, B, Nv] (prune, then attend), all layers in one call."""
        g = self.g
        q0 = g.queries([0], device=self.dev)[0]
        K, V = g.prompt_kv(range(self.L), device=self.dev)
        self.ctx.prefill_select_scored(q0, K, V, g.text_len.tolist(), scores, self.out)
        self.q_cur = q0
        return self.out

    def check_prefill_scored_unit(self, b, l, scores):
        wl, g, s = self.wl, self.g, self.sched
        t0 = wl.sys_len + wl.num_visual + int(g.text_len[b])
        K, V = g.kv_rows([b], [l], range(t0))
        q = g.queries([0], [l])[0, 0, b]
        sc = scores[l, b].double().cpu().numpy()
        ref_out, cache = O.prefill_select_scored(f64(q), f64(K[0, 0]), f64(V[0, 0]), wl.sys_len, wl.num_visual,
                                                 s.n0(l), sc, rank_ordered=self.static)
        assert_out_close(f64(self.out[l, b]), ref_out, wl.dtype, f"scored prefill out b={b} l={l}")
        ids, cnt, mass = self.kept(l)
        n = int(cnt[b])
        assert n == s.n0(l)
        if self.static and n < wl.num_visual:     # layers that are not pruned keep the prompt's order
            assert ids[b, :n].tolist() == cache.ids.tolist()
        else:
            assert sorted(ids[b, :n].tolist()) == sorted(cache.ids.tolist())
        if n < wl.num_visual:
            assert np.array_equal(mass[b], scores[l, b].cpu().numpy())
        self.stats["exact"] += 1
        self.stats["units"] += 1

    def inputs(self, step):
        g = self.g
        if self.overlap:
            # steps that overlap need their inputs complete before the launch ahead of them begins: generate a
            # block of steps, wait for it, then hand the steps out one by one
            if step not in self._ahead:
                steps = list(range(step, min(self.wl.decode_steps, step + 15) + 1))
                q = g.queries(steps, device=self.dev)
                kn, vn = g.new_kv(steps, device=self.dev)
                torch.cuda.synchronize(self.dev)
                self._ahead = {t: (q[i], kn[i], vn[i]) for i, t in enumerate(steps)}
            return self._ahead[step]
        q = g.queries([step], device=self.dev)[0]
        kn, vn = g.new_kv([step], device=self.dev)
        return q, kn[0], vn[0]

    def decode(self, step, layers_per_call=None):
        q, kn, vn = self.inputs(step)
        lpc = layers_per_call or self.L
        for l0 in range(0, self.L, lpc):
            n = min(lpc, self.L - l0)
            self.ctx.decode_step(step, q[l0:l0 + n], kn[l0:l0 + n], vn[l0:l0 + n], self.out[l0:l0 + n],
                                 layer_begin=l0)
        self.q_cur, self.kn_cur, self.vn_cur = q, kn, vn
        return self.out

    def kept(self, layer):
        ids, cnt, mass = self.ctx.get_kept(layer)
        return ids.cpu().numpy(), cnt.cpu().numpy(), mass.cpu().numpy()

    def snapshot(self, layers):
        """{layer: (ids [B, Nv], count [B])} of the current device state."""
        snap = {l: self.kept(l)[:2] for l in layers}
        for l in list(snap):
            src = self.lazy_source(l)
            if src is not None and src not in snap:
                snap[src] = self.kept(src)[:2]
        self._before_all = snap
        return snap

    # ------------------------------------------------------------------ checking
    def lazy_source(self, l):
        """The layer whose q and K layer l inherits (QK heredity), or None."""
        if not (self.lazy_mask >> l) & 1:
            return None
        s = l - 1
        while (self.lazy_mask >> s) & 1:
            s -= 1
        return s

    def stage_head(self, l):
        wl = self.wl
        if not self.shared or l < wl.first_prune_layer:
            return l
        return wl.first_prune_layer + (l - wl.first_prune_layer) // wl.stride * wl.stride

    def _judge_follower(self, b, l, step, ids_before, n, where):
        """A layer that follows its stage's pruning layer holds exactly the pruning layer's rows, in the
        same order, and that set is judged against the pruning layer's oracle scores."""
        src = self.stage_head(l)
        ids, cnt, _ = self.kept(l)
        ids_s, cnt_s, _ = self.kept(src)
        assert int(cnt[b]) == int(cnt_s[b]) == n, where
        assert np.array_equal(ids[b, :n], ids_s[b, :n]), f"{where}: rows differ from the pruning layer's"
        verdict = check_kept(self._src_mass[(b, src, step)], np.asarray(ids_before), n, ids[b, :n])
        self.stats[verdict] += 1
        self.stats["units"] += 1

    def check_prefill_unit(self, b, l):
        wl, g, s = self.wl, self.g, self.sched
        t0 = wl.sys_len + wl.num_visual + int(g.text_len[b])
        K, V = g.kv_rows([b], [l], range(t0))
        q = g.queries([0], [l])[0, 0, b]
        ref_out, ref_mass, _ = O.prefill_select(f64(q), f64(K[0, 0]), f64(V[0, 0]), wl.sys_len, wl.num_visual,
                                                s.n0(l))
        src = self.lazy_source(l)
        if src is not None:     # inherited probabilities: the source's query and keys, this layer's values
            Ks, _ = g.kv_rows([b], [src], range(t0))
            qs = g.queries([0], [src])[0, 0, b]
            ref_out = O.attend_inherited(f64(qs), f64(Ks[0, 0]), f64(V[0, 0]))
        got = f64(self.out[l, b])
        assert_out_close(got, ref_out, wl.dtype, f"prefill out b={b} l={l}")
        ids, cnt, mass = self.kept(l)
        n = int(cnt[b])
        assert n == s.n0(l), (n, s.n0(l))
        if self.stage_head(l) != l:
            self._judge_follower(b, l, 0, np.arange(wl.num_visual), n, f"prefill b={b} l={l}")
            return
        self._src_mass[(b, l, 0)] = ref_mass
        self._judge(ref_mass, np.arange(wl.num_visual), s.n0(l), ids[b, :n], mass[b], trimmed=s.n0(l) < wl.num_visual,
                    where=f"prefill b={b} l={l}")
        if self.static and s.n0(l) < wl.num_visual:
            assert_rank_ordered(ref_mass, ids[b, :n], f"prefill order b={b} l={l}")

    def check_decode_unit(self, b, l, step, before):
        """`before` = (ids [B, Nv], count [B]) of layer l taken before the step ran."""
        wl, g, s = self.wl, self.g, self.sched
        ids_b, cnt_b = before
        nb = int(cnt_b[b])
        cache = rebuild_cache(wl, g, b, l, ids_b[b, :nb], step - 1)
        src = self.lazy_source(l)
        if src is not None:
            assert not self.static
            ids_s, cnt_s = self._before_all[src]
            assert int(cnt_s[b]) == nb and np.array_equal(ids_s[b, :nb], ids_b[b, :nb])
            cache_src = rebuild_cache(wl, g, b, src, ids_s[b, :nb], step - 1)
            kn_s = f64(self.kn_cur[src, b])
            cache_src.K_txt = np.concatenate([cache_src.K_txt, kn_s[:, None, :]], axis=1)
            cache_src.V_txt = np.concatenate([cache_src.V_txt, np.zeros_like(kn_s)[:, None, :]], axis=1)
            head = self.stage_head(l)
            sel = self._src_mass.get((b, head, step)) if head != l else None
            n_t = s.n(l, step)
            if sel is None:
                assert n_t >= nb, "a lazy layer that evicts must follow a pruning layer"
                sel = np.zeros(nb)
            ref_out = O.decode_step_lazy(cache, cache_src, f64(self.q_cur[src, b]), f64(self.vn_cur[l, b]), n_t, sel)
            assert_out_close(f64(self.out[l, b]), ref_out, wl.dtype, f"lazy decode out b={b} l={l} t={step}")
            ids, cnt, _ = self.kept(l)
            n = int(cnt[b])
            assert n == min(nb, n_t)
            if head != l:
                self._judge_follower(b, l, step, ids_b[b, :nb], n, f"lazy decode b={b} l={l} t={step}")
            else:
                assert np.array_equal(ids[b, :n], ids_b[b, :n])
                self.stats["exact"] += 1
                self.stats["units"] += 1
            return
        if self.static:
            ref_out = O.decode_step_static(cache, f64(self.q_cur[l, b]), f64(self.kn_cur[l, b]), f64(self.vn_cur[l, b]),
                                           s.n(l, step))
            assert_out_close(f64(self.out[l, b]), ref_out, wl.dtype, f"static decode out b={b} l={l} t={step}")
            ids, cnt, _ = self.kept(l)
            n = int(cnt[b])
            assert n == min(nb, s.n(l, step))
            assert np.array_equal(ids[b, :n], ids_b[b, :n]), "static-rank cut must keep a prefix of the saved order"
            self.stats["exact"] += 1
            self.stats["units"] += 1
            return
        ref_out, ref_mass, ids_before = O.decode_step(cache, f64(self.q_cur[l, b]), f64(self.kn_cur[l, b]),
                                                      f64(self.vn_cur[l, b]), s.n(l, step))
        assert_out_close(f64(self.out[l, b]), ref_out, wl.dtype, f"decode out b={b} l={l} t={step}")
        ids, cnt, mass = self.kept(l)
        n = int(cnt[b])
        assert n == s.n(l, step) == min(nb, s.n(l, step)), (n, s.n(l, step), nb)
        if self.stage_head(l) != l:
            self._judge_follower(b, l, step, ids_before, n, f"decode b={b} l={l} t={step}")
            return
        self._src_mass[(b, l, step)] = ref_mass
        self._judge(ref_mass, ids_before, n, ids[b, :n], mass[b], trimmed=n < nb, where=f"decode b={b} l={l} t={step}")

    def _judge(self, ref_mass, ids_before, k, got_ids, got_mass_by_id, trimmed, where):
        assert len(set(got_ids.tolist())) == len(got_ids), f"{where}: duplicate ids"
        if trimmed:
            gm = got_mass_by_id[np.asarray(ids_before, dtype=np.int64)]
            assert np.allclose(gm, ref_mass, rtol=MASS_RTOL, atol=MASS_ATOL), \
                f"{where}: mass max rel err {np.max(np.abs(gm - ref_mass) / np.maximum(ref_mass, 1e-12))}"
        verdict = check_kept(ref_mass, np.asarray(ids_before), k, got_ids)
        self.stats[verdict] += 1
        self.stats["units"] += 1

    def check_rows_unit(self, b, l, h, step):
        """Cache rows are bit-identical to the generated rows their ids name; text rows are [S | I | O]."""
        wl, g = self.wl, self.g
        ids, cnt, _ = self.kept(l)
        n = int(cnt[b])
        kv, vv, kt, vt = self.ctx.get_rows(l, b, h)
        text = int(g.text_len[b])
        if n:
            Kr, Vr = g.kv_rows([b], [l], (wl.sys_len + ids[b, :n]).tolist())
            assert torch.equal(kv[:n].cpu(), Kr[0, 0, h]) and torch.equal(vv[:n].cpu(), Vr[0, 0, h])
        toks = list(range(wl.sys_len)) + list(range(wl.sys_len + wl.num_visual, wl.sys_len + wl.num_visual + text)) \
            + [g.gen_token(s) for s in range(1, step + 1)]
        Kt, Vt = g.kv_rows([b], [l], toks)
        assert torch.equal(vt[:len(toks)].cpu(), Vt[0, 0, h])
        nk = len(toks) - step if self.lazy_source(l) is not None else len(toks)   # a lazy layer stores no new keys
        assert torch.equal(kt[:nk].cpu(), Kt[0, 0, h, :nk])


def run_and_check(wl: Workload, steps, check_steps=None, units=None, layers_per_call=None, rows_checks=2,
                  rows_units=None, **cfg):
    """Prefill + decode `steps` steps; check every (b, l) unit (or the sampled `units`) at `check_steps`.
    Cache rows are compared for the first `rows_checks` units, or for `rows_units` if given."""
    run = GpuRun(wl, **cfg)
    try:
        all_units = [(b, l) for l in range(wl.num_layers) for b in range(wl.batch)]
        units = all_units if units is None else units
        check_steps = set(range(0, steps + 1)) if check_steps is None else set(check_steps)
        layers = sorted(set(l for _, l in units))
        run.prefill(layers_per_call)
        if 0 in check_steps:
            for b, l in units:
                run.check_prefill_unit(b, l)
        for t in range(1, steps + 1):
            before = run.snapshot(layers) if t in check_steps else None
            run.decode(t, layers_per_call)
            if t in check_steps:
                for b, l in units:
                    run.check_decode_unit(b, l, t, before[l])
                for b, l in (units[:rows_checks] if rows_units is None else rows_units):
                    run.check_rows_unit(b, l, (t * 7) % wl.num_heads, t)
        assert run.ctx.status() == 0
        return run.stats
    finally:
        run.close()
