"""Behaviour of the C ABI on a GPU beyond plain parity: host-buffer step, call-order errors,
context reuse, bookkeeping queries, profiling counters, schedule variants."""
import numpy as np
import pytest
import torch

from paper_2412_20105_b200 import binding as B
from synth import SynthInputs, get_workload
from gpu_harness import GpuRun, run_and_check
from helpers import make_schedule

pytestmark = pytest.mark.gpu


def _small(**kw):
    base = dict(dtype="bf16", head_dim=128, num_heads=4, num_layers=6, batch=2, sys_len=5, num_visual=200,
                text_len_min=3, text_len_max=20, decode_steps=12, first_prune_layer=2, stride=2,
                step_ratio_bp=1500, tau=12.0, num_planted=10)
    base.update(kw)
    return get_workload("tiny").scaled(**base)


@pytest.mark.parametrize("packed", [False, True])
def test_host_buffer_step_equals_device_step(packed):
    """`packed`: q, k_new, v_new back to back in one pinned buffer (the library's single-copy path);
    otherwise three separate buffers (three copies)."""
    wl = _small()
    a, b = GpuRun(wl), GpuRun(wl)
    try:
        a.prefill(); b.prefill()
        assert torch.equal(a.out, b.out)
        for t in range(1, 6):
            a.decode(t)
            q, kn, vn = b.inputs(t)
            if packed:
                hqkv = torch.stack([q.cpu(), kn.cpu(), vn.cpu()]).contiguous().pin_memory()
                hq, hk, hv = hqkv[0], hqkv[1], hqkv[2]
                assert hk.data_ptr() == hq.data_ptr() + hq.numel() * hq.element_size()
            else:
                hq, hk, hv = (x.cpu().pin_memory() for x in (q, kn, vn))
            hout = torch.empty_like(q.cpu()).pin_memory()
            b.ctx.decode_step_host(t, hq, hk, hv, hout)
            torch.cuda.synchronize()
            assert torch.equal(hout, a.out.cpu()), t
            for l in range(wl.num_layers):
                ia, ca, _ = a.kept(l)
                ib, cb, _ = b.kept(l)
                assert np.array_equal(ca, cb)
                for s in range(wl.batch):
                    assert np.array_equal(ia[s, :ca[s]], ib[s, :cb[s]])
        assert a.ctx.status() == 0 and b.ctx.status() == 0
    finally:
        a.close(); b.close()


@pytest.mark.parametrize("overlap", [False, True])
def test_host_buffer_generation_runs_ahead_of_the_gpu(overlap):
    """Prefill and every decode step through the host-buffer calls, enqueued back to back with no synchronisation
    in between (the library's copy streams run ahead of and behind the kernels), against the same generation
    with device buffers: outputs bit-identical, same kept ids.  st3_host_sync + a wait on the caller's stream
    is all that makes the host outputs readable."""
    wl = _small()
    steps = 9
    a, b = GpuRun(wl), GpuRun(wl, overlap=overlap, host_prefill=1)
    try:
        g = b.g
        q0 = g.queries([0])[0]
        K, V = g.prompt_kv(range(wl.num_layers))
        hq0, hK, hV = q0.pin_memory(), K.pin_memory(), V.pin_memory()
        hout0 = torch.empty_like(hq0).pin_memory()
        qs = g.queries(list(range(1, steps + 1)))
        kn, vn = g.new_kv(list(range(1, steps + 1)))
        hqkv = torch.stack([qs, kn, vn], dim=1).contiguous().pin_memory()        # [step][q | k | v]
        hout = torch.zeros_like(qs).pin_memory()
        b.ctx.prefill_select_host(hq0, hK, hV, g.text_len.tolist(), hout0)
        for t in range(1, steps + 1):
            b.ctx.decode_step_host(t, hqkv[t - 1, 0], hqkv[t - 1, 1], hqkv[t - 1, 2], hout[t - 1])
        b.ctx.host_sync()
        torch.cuda.current_stream().synchronize()
        a.prefill()
        assert torch.equal(hout0, a.out.cpu())
        for t in range(1, steps + 1):
            a.decode(t)
            assert torch.equal(hout[t - 1], a.out.cpu()), t
        for l in range(wl.num_layers):
            ia, ca, _ = a.kept(l)
            ib, cb, _ = b.kept(l)
            assert np.array_equal(ca, cb)
            for s in range(wl.batch):
                assert np.array_equal(ia[s, :ca[s]], ib[s, :cb[s]])
        assert a.ctx.status() == 0 and b.ctx.status() == 0
        # a second generation on the same context reuses the staging areas behind the first one's work
        b.ctx.prefill_select_host(hq0, hK, hV, g.text_len.tolist(), hout0)
        b.ctx.decode_step_host(1, hqkv[0, 0], hqkv[0, 1], hqkv[0, 2], hout[0])
        b.ctx.host_sync()
        torch.cuda.current_stream().synchronize()
        a.prefill(); a.decode(1)
        assert torch.equal(hout[0], a.out.cpu()) and b.ctx.status() == 0
    finally:
        a.close(); b.close()


def test_host_buffer_prefill_needs_its_staging_areas():
    wl = _small()
    run = GpuRun(wl)                       # host_prefill = 0
    try:
        g = run.g
        q0 = g.queries([0])[0].pin_memory()
        K, V = g.prompt_kv(range(wl.num_layers))
        with pytest.raises(B.St3Error) as e:
            run.ctx.prefill_select_host(q0, K.pin_memory(), V.pin_memory(), g.text_len.tolist(),
                                        torch.empty_like(q0).pin_memory())
        assert e.value.code == 3
    finally:
        run.close()


def test_call_order_and_capacity_errors():
    wl = _small()
    run = GpuRun(wl)
    try:
        q, kn, vn = run.inputs(1)
        with pytest.raises(B.St3Error) as e:                      # decode before any prefill
            run.ctx.decode_step(1, q, kn, vn, run.out)
        assert e.value.code == 3
        run.prefill()
        with pytest.raises(B.St3Error) as e:                      # step gap
            run.ctx.decode_step(2, q, kn, vn, run.out)
        assert e.value.code == 3
        run.ctx.decode_step(1, q, kn, vn, run.out)
        with pytest.raises(B.St3Error) as e:                      # same step twice
            run.ctx.decode_step(1, q, kn, vn, run.out)
        assert e.value.code == 3
        with pytest.raises(B.St3Error) as e:                      # beyond max_decode_steps
            run.ctx.decode_step(wl.decode_steps + 1, q, kn, vn, run.out)
        assert e.value.code == 4
        with pytest.raises(B.St3Error) as e:                      # layer range out of bounds
            run.ctx.decode_step(2, q, kn, vn, run.out, layer_begin=1)
        assert e.value.code == 1
        with pytest.raises(B.St3Error) as e:                      # text longer than the configured maximum
            B.st3_prefill_select(run.ctx.handle, 0, wl.num_layers, run.q_cur.data_ptr(), run.q_cur.data_ptr(),
                                 run.q_cur.data_ptr(), [wl.text_len_max + 1] * wl.batch, run.out.data_ptr(), 0)
        assert e.value.code == 4
        with pytest.raises(B.St3Error) as e:                      # misaligned pointer
            B.st3_decode_step(run.ctx.handle, 2, 0, wl.num_layers, q.data_ptr() + 2, kn.data_ptr(), vn.data_ptr(),
                              run.out.data_ptr(), 0)
        assert e.value.code == 1
        # the failed calls changed nothing: step 2 still works and still matches the oracle
        before = run.snapshot(range(wl.num_layers))
        run.decode(2)
        for l in range(wl.num_layers):
            run.check_decode_unit(0, l, 2, before[l])
        assert run.ctx.status() == 0
    finally:
        run.close()


def test_context_is_reusable_for_a_new_generation():
    wl = _small()
    run = GpuRun(wl)
    try:
        run.prefill()
        for t in range(1, 5):
            run.decode(t)
        first = {l: run.kept(l) for l in range(wl.num_layers)}
        out_first = run.out.clone()
        run.prefill()                                             # same prompt again: state starts over
        for t in range(1, 5):
            run.decode(t)
        assert torch.equal(out_first, run.out)
        for l in range(wl.num_layers):
            ids, cnt, _ = run.kept(l)
            assert np.array_equal(cnt, first[l][1])
            for s in range(wl.batch):
                assert np.array_equal(ids[s, :cnt[s]], first[l][0][s, :cnt[s]])
        assert run.ctx.status() == 0
    finally:
        run.close()


def test_rows_held_and_launch_counters_follow_the_schedule():
    wl = _small()
    run = GpuRun(wl)
    try:
        assert run.ctx.rows_held() == (0, 0)
        n0 = run.ctx.launch_count()
        run.prefill()
        assert run.ctx.launch_count() - n0 == 3                   # ingest, attend, finish
        sched = make_schedule(wl)
        text = run.g.text_len
        for t in range(0, 4):
            if t:
                run.decode(t)
            vis, oth = run.ctx.rows_held()
            assert vis == wl.batch * sum(sched.n(l, t) for l in range(wl.num_layers))
            assert oth == wl.num_layers * sum(wl.sys_len + int(x) + t for x in text)
        assert run.ctx.launch_count() - n0 == 3 + 2 * 3
        B.st3_profile_enable(run.ctx.handle, True)
        run.decode(4); run.decode(5)
        a_ms, f_ms, na, nf = B.st3_profile_read(run.ctx.handle)
        assert na == nf == 2 and a_ms > 0 and f_ms > 0
        B.st3_profile_enable(run.ctx.handle, False)
        assert run.ctx.status() == 0
    finally:
        run.close()


@pytest.mark.parametrize("anneal,kw", [("linear", dict(tau=12.0)), ("exp", dict(sigma=4.0)), ("none", dict())])
def test_other_attenuation_functions(anneal, kw):
    code = {"linear": B.ST3_ANNEAL_LINEAR, "exp": B.ST3_ANNEAL_EXP, "none": B.ST3_ANNEAL_NONE}[anneal]
    wl = _small(**{k: v for k, v in kw.items() if k == "tau"})
    stats = run_and_check(wl, wl.decode_steps, sched_kw=dict(anneal=anneal, **{k: v for k, v in kw.items() if k == "sigma"}),
                          anneal=code, **{k: v for k, v in kw.items() if k == "sigma"})
    assert stats["units"] == (wl.decode_steps + 1) * wl.num_layers * wl.batch


def test_layer_by_layer_calls_match_one_call_for_all_layers():
    wl = _small()
    a, b = GpuRun(wl), GpuRun(wl)
    try:
        a.prefill(); b.prefill(layers_per_call=1)
        assert torch.equal(a.out, b.out)
        for t in range(1, 5):
            a.decode(t); b.decode(t, layers_per_call=1)
            assert torch.equal(a.out, b.out), t
        assert a.ctx.status() == 0 and b.ctx.status() == 0
    finally:
        a.close(); b.close()


def _handmade(nv, H=2, D=64, sys_len=2, text=3, steps=4, keep_bp=5000, **cfg_kw):
    cfg = B.make_config(num_layers=1, num_heads=H, head_dim=D, dtype="f32", batch=1, sys_len=sys_len,
                        num_visual=nv, max_text_len=text, max_decode_steps=steps, stride=1, step_ratio_bp=0,
                        first_prune_layer=0, first_ratio_bp=10000 - keep_bp, tau=float(steps), **cfg_kw)
    return cfg, B.Context(cfg)


@pytest.mark.parametrize("static_rank", [0, 1])
def test_equal_scores_keep_the_lowest_original_indices(static_rank):
    """Every visual key identical => every visual score identical: Top must fall back on the index."""
    nv, H, D, sys_len, text = 200, 2, 64, 2, 3
    cfg, ctx = _handmade(nv, H, D, sys_len, text, static_rank=static_rank)
    try:
        g = torch.Generator().manual_seed(5)
        T0 = sys_len + nv + text
        K = torch.randn(1, 1, H, T0, D, generator=g)
        V = torch.randn(1, 1, H, T0, D, generator=g)
        K[:, :, :, sys_len:sys_len + nv] = K[:, :, :, sys_len:sys_len + 1]          # all visual keys alike
        q = torch.randn(1, 1, H, D, generator=g)
        out = torch.empty(1, 1, H, D, device="cuda")
        ctx.prefill_select(q.cuda(), K.cuda(), V.cuda(), [text], out)
        ids, cnt, mass = ctx.get_kept(0)
        n = int(cnt[0])
        assert n == nv // 2
        assert sorted(ids[0, :n].tolist()) == list(range(n))                        # the n lowest indices
        if static_rank:
            assert ids[0, :n].tolist() == list(range(n))                            # and in index order
        m = mass[0].cpu().numpy()
        assert np.all(m == m[0]) and m[0] > 0                                       # bit-identical scores
        # decode steps keep dropping the highest remaining indices
        for t in range(1, 4):
            kn = torch.randn(1, 1, H, D, generator=g).cuda()
            ctx.decode_step(t, q.cuda(), kn, kn, out)
            ids, cnt, _ = ctx.get_kept(0)
            k = B.st3_schedule_count(cfg, 0, t)
            assert int(cnt[0]) == k and sorted(ids[0, :k].tolist()) == list(range(k))
        assert ctx.status() == 0
    finally:
        ctx.close()


def test_two_score_levels_with_ties_at_the_cut():
    """Half of the visual keys get a clearly larger logit; the cut falls inside the lower tie class."""
    nv, H, D, sys_len, text = 96, 2, 64, 1, 2
    cfg, ctx = _handmade(nv, H, D, sys_len, text, keep_bp=7500)
    try:
        g = torch.Generator().manual_seed(6)
        T0 = sys_len + nv + text
        K = torch.randn(1, 1, H, T0, D, generator=g)
        V = torch.randn(1, 1, H, T0, D, generator=g)
        q = torch.randn(1, 1, H, D, generator=g)
        lo, hi = K[:, :, :, sys_len:sys_len + 1].clone(), None
        hi = lo + 0.5 * q[:, :, :, None, :]                                          # larger q.k for every head
        strong = torch.zeros(nv, dtype=torch.bool)
        strong[torch.randperm(nv, generator=g)[:nv // 2]] = True
        K[:, :, :, sys_len:sys_len + nv] = torch.where(strong[None, None, None, :, None], hi, lo)
        out = torch.empty(1, 1, H, D, device="cuda")
        ctx.prefill_select(q.cuda(), K.cuda(), V.cuda(), [text], out)
        ids, cnt, _ = ctx.get_kept(0)
        n = int(cnt[0])
        assert n == 72
        weak_ids = [i for i in range(nv) if not strong[i]]
        want = set(i for i in range(nv) if strong[i]) | set(weak_ids[:72 - 48])      # all strong + lowest weak
        assert set(ids[0, :n].tolist()) == want
        assert ctx.status() == 0
    finally:
        ctx.close()


def test_inputs_from_a_producer_that_signals_completion_early():
    """q, k_new and v_new of every step are written by a kernel that allows its dependents to launch and only
    then, 30 us later, writes them.  In the default mode the step must still see the written values (its
    kernels start only when the producer's grid has finished): the outputs equal those of a run whose inputs
    were in place long before."""
    import native
    lib = native.load()
    wl = _small()
    a, b = GpuRun(wl), GpuRun(wl)
    try:
        a.prefill(); b.prefill()
        st = torch.cuda.current_stream().cuda_stream
        for t in range(1, 6):
            a.decode(t)
            q, kn, vn = b.inputs(t)
            src = torch.stack([q, kn, vn]).contiguous()
            dst = torch.zeros_like(src)                         # stale contents: zeros
            torch.cuda.synchronize()
            n16 = src.numel() * src.element_size() // 16
            assert lib.st3_test_early_trigger_copy(dst.data_ptr(), src.data_ptr(), n16, 30, st) == 0
            b.ctx.decode_step(t, dst[0], dst[1], dst[2], b.out)
            torch.cuda.synchronize()
            assert torch.equal(a.out, b.out), t
            for l in range(wl.num_layers):
                ia, ca, _ = a.kept(l)
                ib, cb, _ = b.kept(l)
                assert np.array_equal(ca, cb) and all(np.array_equal(ia[s, :ca[s]], ib[s, :cb[s]])
                                                      for s in range(wl.batch))
            b.check_rows_unit(0, 1, 0, t)                       # the appended rows are the written ones too
        assert a.ctx.status() == 0 and b.ctx.status() == 0
    finally:
        a.close(); b.close()


def test_a_new_generation_starts_at_layer_zero():
    """Prefilling layer 0 opens a new generation: layers that have not been prefilled again cannot decode."""
    wl = _small()
    run = GpuRun(wl)
    try:
        run.prefill()
        run.decode(1)
        g = run.g
        q0 = g.queries([0], device=run.dev)[0]
        K, V = g.prompt_kv([0, 1], device=run.dev)
        run.ctx.prefill_select(q0[0:2].contiguous(), K, V, g.text_len.tolist(), run.out[0:2], layer_begin=0)
        q, kn, vn = run.inputs(1)
        run.ctx.decode_step(1, q[0:2], kn[0:2], vn[0:2], run.out[0:2], layer_begin=0)     # prefilled again: fine
        with pytest.raises(B.St3Error) as e:                                              # layers 2.. are stale
            run.ctx.decode_step(1, q[2:], kn[2:], vn[2:], run.out[2:], layer_begin=2)
        assert e.value.code == 3
        with pytest.raises(B.St3Error) as e:
            run.ctx.decode_step(2, q[2:], kn[2:], vn[2:], run.out[2:], layer_begin=2)
        assert e.value.code == 3
        assert run.ctx.status() == 0
    finally:
        run.close()
