#!/usr/bin/env python
"""Benchmark of the ST^3 decode-attention + trimming path on synthetic LLaVA-shaped workloads.

One bench "step" is one whole pass of the hot path over one batch: prefill-select of every layer
followed by all decode steps of the workload (append, attend, score, select, compact).  The
metric is decode tokens per second = sequences x decode steps / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle on a bounded sample of
the same workload (see `cpu_baseline.sample` in its line).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from synth import SynthInputs, get_workload

METRIC = "decode-step attn+trim tokens/s at LLaVA-1.5-7B shape"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the attention kernel measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum over
# three launches, see profiles/), as a ratio to the algorithmic bytes of the same launches.  llava15_7b: decode
# steps 43-45.  llava15_7b_b32: captured on a cut of the workload small enough for the profiler (4 of its 32
# sequences, decode steps 5-7); a launch's traffic grows in proportion to its sequences (every sequence brings
# its own rows, nothing is shared), so the ratio carries over to the full batch.  Valid only for the kernel
# source it was taken on: the hash covers csrc/st3_common.cuh and csrc/st3_attend.cuh.
ATTEND_TRAFFIC = {"kernel_sha256": "6241ff7b8dda89b239ff1f76d267d3b0ab0a9ccea2642b25bc1ca30e81b08801",
                  "ratio": {"llava15_7b": 1.015, "llava15_7b_b32": 1.021}}


def attend_kernel_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in ("st3_common.cuh", "st3_attend.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2412_20105_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def attend_traffic_ratio(workload_name):
    try:
        if attend_kernel_sha256() == ATTEND_TRAFFIC["kernel_sha256"]:
            return ATTEND_TRAFFIC["ratio"].get(workload_name)
    except Exception:
        pass
    return None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ----------------------------------------------------------------------------------------------
# algorithmic bytes of the attention kernel
# ----------------------------------------------------------------------------------------------
FOLLOWERS_PER_ITEM = 62  # lazy layers whose values ride on one work item of their source (kMaxFollow in the kernels)


def lazy_offsets(cfg):
    """{layer: k} for every lazy layer: it is the k-th lazy layer above its source (QK heredity, Eq. 6)."""
    out, k = {}, 0
    for l in range(cfg.num_layers):
        k = k + 1 if (cfg.lazy_mask >> l) & 1 else 0
        if k:
            out[l] = k
    return out


def attend_bytes(wl, cfg, B_mod, text_len, step):
    """Bytes the attention kernel of one launch must move (all layers, all sequences).

    Per (sequence, layer): every cached K and V row once (r*T_cur, the newest row read from the
    step's inputs), the newest row written to the cache (r), the query (H*D*e) and, where the
    layer evicts at this step, one fp32 logit per head per visual row (4*H*n_cur).  A lazy layer
    (QK heredity) whose values ride on its source's work items moves its V rows only (r/2 per row,
    no query).
    """
    e = 2 if wl.dtype == "bf16" else 4
    H, D = wl.num_heads, wl.head_dim
    r = 2 * H * D * e
    lazy = lazy_offsets(cfg)
    pruning = lambda l: l if not cfg.stage_shared or l < wl.first_prune_layer else \
        wl.first_prune_layer + (l - wl.first_prune_layer) // wl.stride * wl.stride
    total = 0
    for l in range(wl.num_layers):
        n_cur = wl.num_visual if step == 0 else B_mod.st3_schedule_count(cfg, l, step - 1)
        n_tgt = B_mod.st3_schedule_count(cfg, l, step)
        rides = l in lazy and lazy[l] % (FOLLOWERS_PER_ITEM + 1) != 0
        for b in range(wl.batch):
            t_cur = wl.sys_len + n_cur + int(text_len[b]) + step
            if rides:
                total += (r // 2) * t_cur + (r // 2 if step > 0 else 0)
            elif l in lazy:
                total += r * t_cur + (r // 2 if step > 0 else 0) + H * D * e
            else:
                total += r * t_cur + (r if step > 0 else 0) + H * D * e
            if n_tgt < n_cur and pruning(l) == l:
                total += 4 * H * n_cur
    return total


def path_bytes(wl, cfg, B_mod, text_len):
    """Bytes one whole generation must move, by the method's own accounting (not what the kernels happen to
    touch): per (sequence, layer) and decode step every cached K/V row once (r*T_cur), the new row read and
    written (2r), the query read and the output written (2*H*D*e), and, where the layer evicts at this step,
    one fp32 score term per head per visual row written and read back plus ids and scores ((8H+8)*n_cur) and
    the rows that close the holes read and written (2*r*d for d evicted rows, an upper bound on what hole
    filling moves).  Prefill: the prompt rows read and written into the cache (2*r*T0), read again by the last
    query's attention (r*T0), the same selection terms.  Partials of the split attention are scratch of this
    implementation and are not counted."""
    e = 2 if wl.dtype == "bf16" else 4
    H, D = wl.num_heads, wl.head_dim
    r = 2 * H * D * e
    lazy = lazy_offsets(cfg)
    total = 0
    for step in range(0, wl.decode_steps + 1):
        for l in range(wl.num_layers):
            n_cur = wl.num_visual if step == 0 else B_mod.st3_schedule_count(cfg, l, step - 1)
            n_tgt = min(n_cur, B_mod.st3_schedule_count(cfg, l, step))
            # a lazy layer has no keys and no query of its own (Eq. 6): half the row bytes, output only
            rl, io = (r // 2, H * D * e) if l in lazy else (r, 2 * H * D * e)
            for b in range(wl.batch):
                t_cur = wl.sys_len + n_cur + int(text_len[b]) + step
                total += rl * t_cur + io + (2 * rl if step > 0 else 2 * rl * t_cur)
                if n_tgt < n_cur:
                    total += (8 * H + 8) * n_cur + 2 * rl * (n_cur - n_tgt)
    return total


def schedule_of(wl, **kw):
    """The oracle's schedule object for a workload (used by the CPU legs only)."""
    from oracle import st3_oracle as O
    args = dict(num_layers=wl.num_layers, num_visual=wl.num_visual, stride=wl.stride,
                step_ratio_bp=wl.step_ratio_bp, tau=wl.tau, first_ratio_bp=wl.first_ratio_bp,
                first_prune_layer=wl.first_prune_layer)
    args.update(kw)
    return O.Schedule(**args)


def f64(t):
    return t.detach().to("cpu").to(torch.float64).numpy()


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------
class Job:
    """All device-resident inputs of one workload plus a library context."""

    def __init__(self, wl, device, disable_trim=False, rows_per_chunk=0, static_rank=False, stage_shared=False,
                 lazy_mask=0, host_prefill=False):
        from paper_2412_20105_b200 import binding as B
        from paper_2412_20105_b200.build import build
        build()
        self.B = B
        self.wl, self.dev = wl, device
        self.g = SynthInputs(wl)
        self.cfg = B.config_from_workload(wl, disable_trim=int(disable_trim), rows_per_chunk=rows_per_chunk,
                                           static_rank=int(static_rank), stage_shared=int(stage_shared),
                                           lazy_mask=int(lazy_mask), host_prefill=int(host_prefill))
        self.ctx = B.Context(self.cfg, device)
        # every input of a generation is in device memory before its first launch, which is what the
        # overlapping-steps mode asks of its caller
        B.st3_set_overlap(self.ctx.handle, True)
        self.lib = B.load()
        L, T = wl.num_layers, wl.decode_steps
        g = self.g
        self.q0 = g.queries([0], device=device)[0].contiguous()
        Ks, Vs = [], []
        for l in range(L):
            K, V = g.prompt_kv([l], device=device)
            Ks.append(K); Vs.append(V)
        self.K, self.V = torch.cat(Ks), torch.cat(Vs)
        del Ks, Vs
        chunk = 32
        qs, ks, vs = [], [], []
        for s0 in range(1, T + 1, chunk):
            steps = list(range(s0, min(T, s0 + chunk - 1) + 1))
            qs.append(g.queries(steps, device=device))
            kn, vn = g.new_kv(steps, device=device)
            ks.append(kn); vs.append(vn)
        self.q, self.kn, self.vn = torch.cat(qs), torch.cat(ks), torch.cat(vs)        # [T, L, B, H, D]
        self.out = torch.empty_like(self.q)
        self.out0 = torch.empty_like(self.q0)
        self.io_bytes = self.q0.numel() * self.q0.element_size()
        self.text = g.text_len.tolist()
        self.stream = torch.cuda.current_stream(device).cuda_stream

    def generation(self):
        """prefill-select + every decode step, device-resident inputs."""
        B, h, L, st = self.B, self.ctx.handle, self.wl.num_layers, self.stream
        B.st3_prefill_select(h, 0, L, self.q0.data_ptr(), self.K.data_ptr(), self.V.data_ptr(), self.text,
                             self.out0.data_ptr(), st)
        q, k, v, o, nb = self.q.data_ptr(), self.kn.data_ptr(), self.vn.data_ptr(), self.out.data_ptr(), self.io_bytes
        step_fn = self.lib.st3_decode_step
        for t in range(1, self.wl.decode_steps + 1):
            off = (t - 1) * nb
            rc = step_fn(h, t, 0, L, q + off, k + off, v + off, o + off, st)
            if rc:
                raise B.St3Error(rc, f"st3_decode_step t={t}")

    def prefill_only(self):
        self.B.st3_prefill_select(self.ctx.handle, 0, self.wl.num_layers, self.q0.data_ptr(), self.K.data_ptr(),
                                  self.V.data_ptr(), self.text, self.out0.data_ptr(), self.stream)

    def generation_per_layer(self):
        """The calling pattern of a real model: one call per layer, prefill and every decode step."""
        B, h, L, st = self.B, self.ctx.handle, self.wl.num_layers, self.stream
        lb0 = self.q0[0].numel() * self.q0.element_size()                 # bytes of one layer of q / out
        kvb = self.K[0].numel() * self.K.element_size()
        for l in range(L):
            B.st3_prefill_select(h, l, 1, self.q0.data_ptr() + l * lb0, self.K.data_ptr() + l * kvb,
                                 self.V.data_ptr() + l * kvb, self.text, self.out0.data_ptr() + l * lb0, st)
        q, k, v, o, nb = self.q.data_ptr(), self.kn.data_ptr(), self.vn.data_ptr(), self.out.data_ptr(), self.io_bytes
        step_fn = self.lib.st3_decode_step
        for t in range(1, self.wl.decode_steps + 1):
            off = (t - 1) * nb
            for l in range(L):
                o2 = off + l * lb0
                rc = step_fn(h, t, l, 1, q + o2, k + o2, v + o2, o + o2, st)
                if rc:
                    raise B.St3Error(rc, f"st3_decode_step t={t} l={l}")

    def rows_held_curve(self, points=9):
        """(step, visual rows, other rows, K/V bytes held) along one generation: host bookkeeping."""
        wl, B, h = self.wl, self.B, self.ctx.handle
        e = 2 if wl.dtype == "bf16" else 4
        row_bytes = 2 * wl.num_heads * wl.head_dim * e
        want = sorted(set(int(round(x)) for x in np.linspace(0, wl.decode_steps, points)))
        self.prefill_only()
        out = []
        q, k, v, o, nb = self.q.data_ptr(), self.kn.data_ptr(), self.vn.data_ptr(), self.out.data_ptr(), self.io_bytes
        for t in range(0, wl.decode_steps + 1):
            if t:
                off = (t - 1) * nb
                B.st3_decode_step(h, t, 0, wl.num_layers, q + off, k + off, v + off, o + off, self.stream)
            if t in want:
                vis, oth = B.st3_rows_held(h)
                full = wl.batch * wl.num_layers * wl.num_visual
                out.append({"step": t, "visual_rows": vis, "other_rows": oth, "kv_bytes": (vis + oth) * row_bytes,
                            "kv_bytes_untrimmed": (full + oth) * row_bytes})
        return out

    def kept_set_curve(self, points=5):
        """Diagnostics read from the kept-id sets along one generation, averaged over the pruning layers of
        sequence 0: (a) Eq. 10 applied to the kept sets, the share of the tokens held after decode step 1 that
        are still held after step n (the path only ever evicts, so this is how fast the first step's set is
        used up); (b) the share of the planted attentive tokens (or of the kept slots, if fewer) that the kept
        set holds, i.e. whether what is kept is what the synthetic queries attend to."""
        wl, B, h = self.wl, self.B, self.ctx.handle
        layers = [l for l in range(wl.first_prune_layer, wl.num_layers)]
        want = sorted(set(int(round(x)) for x in np.linspace(1, wl.decode_steps, points)))
        self.prefill_only()
        q, k, v, o, nb = self.q.data_ptr(), self.kn.data_ptr(), self.vn.data_ptr(), self.out.data_ptr(), self.io_bytes
        first, out = {}, []
        for t in range(1, wl.decode_steps + 1):
            off = (t - 1) * nb
            B.st3_decode_step(h, t, 0, wl.num_layers, q + off, k + off, v + off, o + off, self.stream)
            if t not in want:
                continue
            ov, rec = [], []
            for l in layers:
                ids, cnt, _ = self.ctx.get_kept(l, with_mass=False)
                kept = set(ids[0, :int(cnt[0])].tolist())
                if t == 1:
                    first[l] = kept
                planted = set(int(i) for i in self.g.planted(0, l))
                ov.append(len(kept & first[l]) / max(1, len(first[l])))
                if kept:
                    rec.append(len(kept & planted) / min(len(planted), len(kept)))
            out.append({"step": t, "overlap_with_step_1": float(np.mean(ov)),
                        "planted_recall": float(np.mean(rec)) if rec else None})   # None: nothing is held any more
        return out

    def make_host(self):
        """Every input of a generation in pinned host memory, and pinned buffers for every output."""
        self.hK, self.hV = self.K.cpu().pin_memory(), self.V.cpu().pin_memory()
        self.hq0 = self.q0.cpu().pin_memory()
        # one pinned buffer [step][q | k_new | v_new]: the three inputs of a step lie back to back, which lets the
        # library bring them over in one copy
        self.hqkv = torch.stack([self.q.cpu(), self.kn.cpu(), self.vn.cpu()], dim=1).contiguous().pin_memory()
        self.hq = self.hqkv[:, 0]
        self.hout = torch.empty_like(self.hq).pin_memory()
        self.hout0 = torch.empty_like(self.hq0).pin_memory()

    def generation_host(self):
        """Same work through the host-buffer calls of the C ABI: every input starts in pinned host memory and
        every output ends there (the context was created with host_prefill = 1)."""
        B, h, L, st = self.B, self.ctx.handle, self.wl.num_layers, self.stream
        B.st3_prefill_select_host(h, 0, L, self.hq0.data_ptr(), self.hK.data_ptr(), self.hV.data_ptr(), self.text,
                                  self.hout0.data_ptr(), st)
        base, o, nb = self.hqkv.data_ptr(), self.hout.data_ptr(), self.io_bytes
        step_fn = self.lib.st3_decode_step_host
        for t in range(1, self.wl.decode_steps + 1):
            off = (t - 1) * nb
            q = base + 3 * off
            rc = step_fn(h, t, 0, L, q, q + nb, q + 2 * nb, o + off, st)
            if rc:
                raise B.St3Error(rc, f"st3_decode_step_host t={t}")
        B.st3_host_sync(h, st)

    def host_pipeline(self, n):
        """n generations through the host-buffer calls on TWO library contexts and two streams, alternating: the
        prompt of generation g+1 crosses the bus (and is ingested and trimmed) while generation g decodes.  The
        inputs are the same pinned buffers for both; each context has its own output buffers.  Forks from and
        joins the current stream, so events around the call time all of it."""
        B, L = self.B, self.wl.num_layers
        if not hasattr(self, "pipe"):
            second = B.Context(self.cfg, self.dev)
            B.st3_set_overlap(second.handle, True)
            self.pipe = [(self.ctx, torch.cuda.Stream(self.dev), self.hout, self.hout0),
                         (second, torch.cuda.Stream(self.dev), torch.empty_like(self.hout).pin_memory(),
                          torch.empty_like(self.hout0).pin_memory())]
        cur = torch.cuda.current_stream(self.dev)
        for _, s, _, _ in self.pipe:
            s.wait_stream(cur)
        base, nb = self.hqkv.data_ptr(), self.io_bytes
        step_fn = self.lib.st3_decode_step_host
        for g in range(n):
            ctx, s, hout, hout0 = self.pipe[g & 1]
            h, st, o = ctx.handle, s.cuda_stream, hout.data_ptr()
            B.st3_prefill_select_host(h, 0, L, self.hq0.data_ptr(), self.hK.data_ptr(), self.hV.data_ptr(), self.text,
                                      hout0.data_ptr(), st)
            for t in range(1, self.wl.decode_steps + 1):
                off = (t - 1) * nb
                q = base + 3 * off
                rc = step_fn(h, t, 0, L, q, q + nb, q + 2 * nb, o + off, st)
                if rc:
                    raise B.St3Error(rc, f"st3_decode_step_host t={t}")
            B.st3_host_sync(h, st)
        for _, s, _, _ in self.pipe:
            cur.wait_stream(s)

    def h2d_bytes(self):
        kv = 2 * self.K.numel() * self.K.element_size()
        return kv + self.io_bytes + 3 * self.io_bytes * self.wl.decode_steps

    def d2h_bytes(self):
        return self.io_bytes * (self.wl.decode_steps + 1)


def timed(fn, n, dist):
    """Device time of n calls of fn in ms (CUDA events on the current stream, max over ranks)."""
    torch.cuda.synchronize()
    if dist:
        torch.distributed.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize()
    if dist:
        torch.distributed.barrier()
    return max_over_ranks(e0.elapsed_time(e1), dist, "cuda")


def max_over_ranks(value, dist, device):
    """The slowest rank's time: what a multi-GPU number is reported on."""
    if not dist:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def replica_workload(wl, rank, world):
    """Replicas work on different data: rank r of a multi-GPU run uses seed + 1000 r."""
    return wl if world == 1 else wl.scaled(seed=wl.seed + 1000 * rank)


def job_value(tokens_per_gen, steps, world, ms):
    """Whole-job tokens/s: every rank processed tokens_per_gen * steps tokens in `ms` (max over ranks)."""
    return world * tokens_per_gen * steps / (ms * 1e-3)


def oracle_sample(wl, g, K, V, q0, q, kn, vn, nsteps, warm_steps, reps=1):
    """Times the oracle, as it stands, on decode steps 1..nsteps of the workload (all layers, all
    sequences, free-running after its own prefill).  Returns (tokens/s, seconds, threads)."""
    from oracle import st3_oracle as O
    sched = schedule_of(wl)
    caches = {}
    for l in range(wl.num_layers):
        for b in range(wl.batch):
            t0 = wl.sys_len + wl.num_visual + int(g.text_len[b])
            _, _, caches[(b, l)] = O.prefill_select(f64(q0[l, b]), f64(K[l, b][:, :t0]), f64(V[l, b][:, :t0]),
                                                    wl.sys_len, wl.num_visual, sched.n0(l))

    def run(t):
        for l in range(wl.num_layers):
            for b in range(wl.batch):
                O.decode_step(caches[(b, l)], f64(q[t - 1, l, b]), f64(kn[t - 1, l, b]), f64(vn[t - 1, l, b]),
                              sched.n(l, t))

    t = 1
    for _ in range(warm_steps):
        run(t); t += 1
    t_start = time.perf_counter()
    first = t
    for _ in range(nsteps):
        run(t); t += 1
    secs = time.perf_counter() - t_start
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = 1
    return wl.batch * nsteps / secs, secs, threads, first, t - 1


def free_running_report(wl, device, steps=None, rel=1e-3):
    """Oracle and GPU run the same generation side by side WITHOUT the oracle ever adopting the GPU's state.
    After prefill and after every decode step the kept visual ids of every (sequence, layer) unit are compared
    as sets.  Reports the first step at which some unit's set differs (None if never), whether the oracle's
    scores at that cut were a near-tie (gap at the boundary <= rel * |s_k|), how many units have left the
    oracle's trajectory by the end, and the largest output error over the units that still agree (absolute
    for fp32, relative to max(|ref|, 1e-2) for bf16)."""
    from oracle import st3_oracle as O
    from paper_2412_20105_b200 import binding as B
    T = wl.decode_steps if steps is None else min(steps, wl.decode_steps)
    g = SynthInputs(wl)
    sched = schedule_of(wl)
    cfg = B.config_from_workload(wl)
    ctx = B.Context(cfg, device)
    L, Bn = wl.num_layers, wl.batch
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    out = torch.empty((L, Bn, wl.num_heads, wl.head_dim), dtype=tdt, device=device)
    text = g.text_len.tolist()
    caches, agree = {}, {}
    first, diverged, max_err = None, 0, 0.0

    def err_of(got, ref):
        if wl.dtype == "f32":
            return float(np.abs(got - ref).max())
        return float((np.abs(got - ref) / np.maximum(np.abs(ref), 1e-2)).max())

    def compare(step, masses, ids_before, ref_out):
        nonlocal first, diverged, max_err
        got_out = f64(out)
        for l in range(L):
            ids, cnt, _ = ctx.get_kept(l, with_mass=False)
            ids, cnt = ids.cpu().numpy(), cnt.cpu().numpy()
            for b in range(Bn):
                if not agree[(b, l)]:
                    continue
                max_err = max(max_err, err_of(got_out[l, b], ref_out[(b, l)]))
                c = caches[(b, l)]
                if set(ids[b, :int(cnt[b])].tolist()) == set(c.ids.tolist()):
                    continue
                agree[(b, l)] = False
                diverged += 1
                if first is None:
                    k = c.n_cur
                    s_k, s_k1 = O.boundary_scores(masses[(b, l)], ids_before[(b, l)], k)
                    gap = None if s_k is None or s_k1 is None else (s_k - s_k1) / max(abs(s_k), 1e-300)
                    first = {"step": step, "layer": l, "sequence": b, "near_tie": gap is not None and gap <= rel,
                             "relative_gap_at_cut": gap}

    try:
        q0 = g.queries([0], device=device)[0]
        masses, before, ref_out = {}, {}, {}
        for l in range(L):
            K, V = g.prompt_kv([l], device=device)
            ctx.prefill_select(q0[l:l + 1].contiguous(), K, V, text, out[l:l + 1], layer_begin=l)
            Kc, Vc, qc = K.cpu(), V.cpu(), q0[l].cpu()
            for b in range(Bn):
                t0 = wl.sys_len + wl.num_visual + int(text[b])
                o, m, caches[(b, l)] = O.prefill_select(f64(qc[b]), f64(Kc[0, b][:, :t0]), f64(Vc[0, b][:, :t0]),
                                                        wl.sys_len, wl.num_visual, sched.n0(l))
                agree[(b, l)] = True
                masses[(b, l)], before[(b, l)], ref_out[(b, l)] = m, np.arange(wl.num_visual), o
        compare(0, masses, before, ref_out)
        for t in range(1, T + 1):
            q = g.queries([t], device=device)[0]
            kn, vn = g.new_kv([t], device=device)
            ctx.decode_step(t, q, kn[0], vn[0], out)
            qc, kc, vc = f64(q), f64(kn[0]), f64(vn[0])
            for l in range(L):
                for b in range(Bn):
                    if agree[(b, l)]:
                        ref_out[(b, l)], masses[(b, l)], before[(b, l)] = O.decode_step(
                            caches[(b, l)], qc[l, b], kc[l, b], vc[l, b], sched.n(l, t))
            compare(t, masses, before, ref_out)
        ctx.status()
    finally:
        ctx.close()
    return {"workload": wl.name, "steps_compared": T, "units": L * Bn, "first_divergence": first,
            "units_diverged_by_the_end": diverged, "max_output_error_while_in_agreement": max_err,
            "error_kind": "max-abs" if wl.dtype == "f32" else "max relative to max(|ref|, 1e-2)",
            "mode": "neither side is re-seeded from the other; kept-id sets compared after every step"}


def prefill_attend_leg(wl, device, iters=10, max_instances=2048):
    """Causal prompt attention (the step before the hot path) on the tensor cores: every layer's
    (sequence, head) instances of the workload in one call, full prompt length."""
    from paper_2412_20105_b200 import binding as B
    if wl.dtype != "bf16" or wl.head_dim != 128:
        return None
    T = wl.sys_len + wl.num_visual + wl.text_len_max
    n = max(wl.num_heads, min(wl.num_layers * wl.batch * wl.num_heads, max_instances))
    n -= n % wl.num_heads
    g = torch.Generator().manual_seed(wl.seed)
    mk = lambda: torch.randn(n, T, 128, generator=g).to(torch.bfloat16).to(device)
    q, k, v = mk(), mk(), mk()
    out = torch.empty_like(q)
    probs = torch.zeros(n, wl.num_visual, device=device)
    scores = torch.zeros(n // wl.num_heads, wl.num_visual, device=device)
    st = torch.cuda.current_stream(device).cuda_stream
    call = lambda: B.st3_prefill_attend(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), probs.data_ptr(),
                                        scores.data_ptr(), None, n, wl.num_heads, T, 128, "bf16", wl.sys_len,
                                        wl.num_visual, st)
    for _ in range(3):
        call()
    ms = timed(call, iters, False) / iters
    flops = n * 4 * 128 * T * (T + 1) / 2          # two GEMMs over the causal half
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, src = float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        peak, src = 1590.0, "fallback"
    tf = flops / (ms * 1e-3) / 1e12
    return {"instances": n, "seq_len": T, "ms": ms, "bound": "tensor", "achieved": tf, "peak": peak,
            "unit": "TFLOP/s", "frac": tf / peak, "peak_source": f"of {src}",
            "flops": "causal half of Q K^T and P V (4 D T (T+1)/2 per instance)"}


def kernel_roofline(job, steps, world):
    """Attention-kernel time from the library's own events (which serialise the launches), against the
    algorithmic bytes of the same launches."""
    B, wl = job.B, job.wl
    B.st3_profile_enable(job.ctx.handle, True)
    for _ in range(steps):
        job.generation()
    attn_ms, finish_ms, n_attn, _ = B.st3_profile_read(job.ctx.handle)
    B.st3_profile_enable(job.ctx.handle, False)
    alg = sum(attend_bytes(wl, job.cfg, B, job.text, t) for t in range(0, wl.decode_steps + 1)) * steps
    peak, peak_kind = measured_peak()
    achieved = alg / (attn_ms * 1e-3) / 1e9
    ratio = attend_traffic_ratio(wl.name) if world == 1 and not job.cfg.lazy_mask else None
    return {"bound": "hbm", "kernel": "st3_attend_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": f"of {peak_kind}",
            "traffic": None if ratio is None else ratio * alg / max(1, n_attn),
            "algorithmic_bytes_per_launch": alg / max(1, n_attn), "us_per_launch": attn_ms * 1e3 / max(1, n_attn),
            "timing_mode": "launches serialised by the events around each kernel (no overlap between a step's "
                           "selection kernel and the next step's attention kernel), so us_per_launch x launches "
                           "exceeds ms_per_step, which is timed with the steps overlapping",
            "launches_timed": n_attn, "attend_share_of_kernel_time": attn_ms / max(1e-9, attn_ms + finish_ms)}


def add_path_fraction(roofline, job, ms_per_generation):
    """Whole fused path: the method's bytes of one generation over its measured time, against the same peak."""
    pb = path_bytes(job.wl, job.cfg, job.B, job.text)
    roofline["path_algorithmic_bytes_per_step"] = pb
    roofline["path_achieved"] = pb / (ms_per_generation * 1e-3) / 1e9
    roofline["path_frac"] = roofline["path_achieved"] / roofline["peak"]
    return roofline


def per_layer_leg(job, n):
    """One library call per layer (the calling pattern of a real decoder): tokens/s, GPU time per call, and the
    host time one st3_decode_step(layer_count=1) call takes (wall clock around a generation's calls, which
    only enqueue work; the queue is drained before and after)."""
    wl = job.wl
    job.generation_per_layer()
    ms = timed(job.generation_per_layer, n, False)
    job.ctx.status()
    calls = wl.num_layers * (wl.decode_steps + 1)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    job.generation_per_layer()
    host_s = time.perf_counter() - t0
    torch.cuda.synchronize()
    job.ctx.status()
    return {"value": wl.batch * wl.decode_steps * n / (ms * 1e-3), "unit": UNIT, "calls_per_generation": calls,
            "gpu_us_per_call": ms * 1e3 / (n * calls), "host_us_per_call": host_s * 1e6 / calls,
            "host_note": "includes the ctypes call overhead of this benchmark's Python loop"}


def qk_heredity_line(wl, device, args, name, mask):
    """One configuration with stage-shared kept sets and the given lazy layers: tokens/s, the attention
    kernel's algorithmic bytes per launch (lazy layers count their V rows only) and its fraction of the peak."""
    job = Job(wl, device, stage_shared=True, lazy_mask=mask, rows_per_chunk=args.rows_per_chunk)
    try:
        for _ in range(3):
            job.generation()
        ms = timed(job.generation, args.steps, False)
        job.ctx.status()
        roof = kernel_roofline(job, 1, 1)
        return {"lazy_layers": name, "value": wl.batch * wl.decode_steps * args.steps / (ms * 1e-3), "unit": UNIT,
                "algorithmic_bytes_per_launch": roof["algorithmic_bytes_per_launch"],
                "us_per_launch": roof["us_per_launch"], "frac": roof["frac"]}
    finally:
        job.ctx.close()
        del job
        torch.cuda.empty_cache()


def other_workload_line(name, device, rank):
    """One timed generation of another LLaVA-shaped workload (after one warm-up generation): tokens/s, the
    attention kernel's and the whole path's fraction of the HBM peak, clocks during the timed generation."""
    wl = get_workload(name)
    job = Job(wl, device)
    try:
        job.generation()
        job.ctx.status()
        sampler = ClockSampler(rank)
        sampler.start()
        time.sleep(0.2)
        ms = timed(job.generation, 1, False)
        clocks = sampler.stop()
        job.ctx.status()
        roof = add_path_fraction(kernel_roofline(job, 1, 1), job, ms)
        return {"workload": wl.name, "value": wl.batch * wl.decode_steps / (ms * 1e-3), "unit": UNIT,
                "ms_per_step": ms, "steps": 1, "warmup": 1, "frac": roof["frac"], "path_frac": roof["path_frac"],
                "achieved": roof["achieved"], "us_per_launch": roof["us_per_launch"], "traffic": roof["traffic"],
                "clocks": clocks}
    finally:
        job.ctx.close()
        del job
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llava15_7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows-per-chunk", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="run a cut of the workload with this many sequences")
    ap.add_argument("--decode-steps", type=int, default=0, help="... and this many decode steps (tau unchanged)")
    ap.add_argument("--stage-shared", action="store_true",
                    help="layers between two pruning layers keep the pruning layer's tokens (strided pruning)")
    ap.add_argument("--lazy-mask", type=lambda x: int(x, 0), default=0,
                    help="bit l set: layer l is lazy (QK heredity); needs --stage-shared inside a pruning stage")
    ap.add_argument("--no-extras", action="store_true", help="skip the e2e, unpruned and cpu_baseline legs")
    ap.add_argument("--e2e-only", action="store_true", help="after the timed run, only the end-to-end leg")
    ap.add_argument("--no-others", action="store_true", help="skip the one-generation runs of the other workloads")
    ap.add_argument("--leg", default="", choices=["", "prefill_attend", "qk_heredity", "per_layer"],
                    help="run one auxiliary leg alone and print its JSON (for timing or profiling that kernel)")
    ap.add_argument("--instances", type=int, default=2048, help="cap on the (sequence, head) instances of --leg")
    args = ap.parse_args()
    wl = get_workload(args.workload)
    if args.batch or args.decode_steps:   # a cut of a workload (for profiler captures that must stay small)
        wl = wl.scaled(name=f"{wl.name}[batch={args.batch or wl.batch},steps={args.decode_steps or wl.decode_steps}]",
                       batch=args.batch or wl.batch, decode_steps=args.decode_steps or wl.decode_steps)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    config = {"workload": f"{wl.name}: B={wl.batch} L={wl.num_layers} H={wl.num_heads} D={wl.head_dim} "
                          f"{wl.dtype}, prompt {wl.sys_len}+{wl.num_visual}+[{wl.text_len_min},{wl.text_len_max}], "
                          f"{wl.decode_steps} decode steps, S={wl.stride} R={wl.step_ratio_bp}bp "
                          f"P={wl.first_ratio_bp}bp tau={wl.tau:g}",
              "step": "prefill-select of all layers + all decode steps of one batch",
              "launch_mode": "one call per decode step over all layers; consecutive steps overlap on the GPU "
                             "(st3_set_overlap: every input is in device memory before the generation starts)",
              "l2": "inputs larger than L2 (per-step K/V working set > 126 MB); no explicit flush",
              "parallelism": f"{args.gpus} independent replica(s), no collectives"}

    if args.impl == "reference":
        if rank != 0:
            return
        g = SynthInputs(wl)
        s_per = 4 if wl.batch == 1 else 1
        n_timed, n_warm = args.steps * s_per, max(1, args.warmup) * s_per
        need = n_timed + n_warm
        L = wl.num_layers
        q0 = g.queries([0])[0]
        Ks, Vs = zip(*[g.prompt_kv([l]) for l in range(L)])
        K, V = torch.cat(Ks), torch.cat(Vs)
        steps = list(range(1, need + 1))
        q = g.queries(steps)
        kn, vn = g.new_kv(steps)
        val, secs, threads, s_first, s_last = oracle_sample(wl, g, K, V, q0, q, kn, vn, n_timed, n_warm)
        sample = (f"oracle (numpy fp64), all {L} layers x {wl.batch} sequence(s), decode steps {s_first}-{s_last} of "
                  f"{wl.decode_steps} after its own prefill; one bench step = {s_per} decode step(s)")
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs * 1e3 / args.steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": config,
                "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                                 "threads": f"numpy fp64; the Python loop over (layer, sequence) is serial, the "
                                            f"matrix products inside it use a BLAS pool of {threads} thread(s)"},
                "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dist = world > 1
    torch.cuda.set_device(local)
    device = torch.device(f"cuda:{local}")
    if args.leg == "prefill_attend":
        if rank == 0:
            print(json.dumps({"leg": args.leg, "workload": wl.name,
                              **(prefill_attend_leg(wl, device, max(1, args.steps), args.instances) or {})}))
        return
    if args.leg == "qk_heredity":
        if rank == 0:
            print(json.dumps({"leg": args.leg, "workload": wl.name, "lines": [
                qk_heredity_line(wl, device, args, name, mask) for name, mask in (
                    ("stage_shared, no lazy layer", 0), ("layers 29-30 inherit layer 28", (1 << 29) | (1 << 30)),
                    ("layers 4-6 inherit layer 3, layers 8-9 inherit layer 7", sum(1 << l for l in (4, 5, 6, 8, 9))))]}))
        return
    if args.leg == "per_layer":
        if rank == 0:
            job = Job(wl, device, rows_per_chunk=args.rows_per_chunk)
            print(json.dumps({"leg": args.leg, "workload": wl.name, **per_layer_leg(job, max(1, args.steps))}))
            job.ctx.close()
        return
    if dist:
        torch.distributed.init_process_group("nccl", device_id=device)
    wl = replica_workload(wl, rank, world)
    job = Job(wl, device, rows_per_chunk=args.rows_per_chunk, stage_shared=args.stage_shared, lazy_mask=args.lazy_mask)
    if args.stage_shared or args.lazy_mask:
        config["variant"] = f"stage_shared={int(args.stage_shared)} lazy_mask={args.lazy_mask:#x}"
    B = job.B
    tokens_per_gen = wl.batch * wl.decode_steps

    for _ in range(max(3, args.warmup)):
        job.generation()
    job.ctx.status()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    n0 = job.ctx.launch_count()
    ms = timed(job.generation, args.steps, dist)
    launches = job.ctx.launch_count() - n0
    clocks = sampler.stop() if rank == 0 else None
    job.ctx.status()
    value = job_value(tokens_per_gen, args.steps, world, ms)

    # per-kernel time of the attention kernel (events around it inside the library), same work
    roofline = add_path_fraction(kernel_roofline(job, args.steps, world), job, ms / args.steps)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic", "config": config,
            "gpu_launches": int(launches), "roofline": roofline, "clocks": clocks}

    # end to end: every input starts in pinned host memory, every output ends there
    if not args.no_extras:
        hjob = Job(wl, device, rows_per_chunk=args.rows_per_chunk, stage_shared=args.stage_shared,
                   lazy_mask=args.lazy_mask, host_prefill=True)
        hjob.make_host()
        for _ in range(2):
            hjob.generation_host()
        ms_one = timed(hjob.generation_host, args.steps, dist)
        hjob.ctx.status()
        # two contexts, alternating: a batch's prompt crosses the bus while the batch before it decodes
        n_pipe = max(8, args.steps)   # enough batches for the pipeline's fill (the first prompt overlaps nothing) to weigh little
        hjob.host_pipeline(2)
        ms_e2e = timed(lambda: hjob.host_pipeline(n_pipe), 1, dist) * args.steps / n_pipe
        for ctx, _, _, _ in hjob.pipe:
            ctx.status()
        line["e2e"] = {"value": job_value(tokens_per_gen, args.steps, world, ms_e2e), "unit": UNIT,
                       "h2d_bytes_per_step": hjob.h2d_bytes(), "d2h_bytes_per_step": hjob.d2h_bytes(),
                       "ms_per_step": ms_e2e / args.steps,
                       "api": "st3_prefill_select_host + st3_decode_step_host + st3_host_sync: pinned host buffers, "
                              "the library's two copy streams run ahead of and behind the kernels; consecutive batches "
                              "alternate between two library contexts on two streams, so that a batch's prompt is "
                              "copied, ingested and trimmed while the batch before it decodes",
                       "generations_timed": n_pipe,
                       "one_context": {"value": job_value(tokens_per_gen, args.steps, world, ms_one),
                                       "ms_per_step": ms_one / args.steps,
                                       "note": "one batch after the other on one context: the prompt's copy overlaps "
                                               "nothing of the batch before it"}}
        hjob.pipe[1][0].close()
        hjob.ctx.close()
        del hjob
        torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_extras and not args.e2e_only:
        # the same kernels with trimming disabled (full KV cache)
        full = Job(wl, device, disable_trim=True, rows_per_chunk=args.rows_per_chunk)
        for _ in range(3):
            full.generation()
        ms_full = timed(full.generation, args.steps, False)
        full.ctx.status()
        v_full = tokens_per_gen * args.steps / (ms_full * 1e-3)
        line["unpruned"] = {"value": v_full, "unit": UNIT, "speedup_from_trimming": value / v_full}
        full.ctx.close()
        del full
        # Algorithm 3 as printed: kept rows in top-index order, decode cuts a prefix (no re-scoring)
        stat = Job(wl, device, static_rank=True, rows_per_chunk=args.rows_per_chunk)
        for _ in range(3):
            stat.generation()
        ms_stat = timed(stat.generation, args.steps, False)
        stat.ctx.status()
        line["static_rank"] = {"value": tokens_per_gen * args.steps / (ms_stat * 1e-3), "unit": UNIT}
        stat.ctx.close()
        del stat
        # QK heredity (Eq. 6): lazy layers move their V rows only.  Stage-shared kept sets with no lazy layer,
        # with the paper's pattern inside the last full stage, and with lazy layers inside the first stage.
        if wl.name == "llava15_7b":
            line["qk_heredity"] = [qk_heredity_line(wl, device, args, name, mask) for name, mask in (
                ("stage_shared, no lazy layer", 0),
                ("layers 29-30 inherit layer 28", (1 << 29) | (1 << 30)),
                ("layers 4-6 inherit layer 3, layers 8-9 inherit layer 7", sum(1 << l for l in (4, 5, 6, 8, 9))))]
        # prefill-select alone, the one-call-per-layer pattern, and K/V held along a generation
        ms_pre = timed(job.prefill_only, args.steps, False)
        line["prefill_select_ms"] = ms_pre / args.steps
        line["per_layer_calls"] = per_layer_leg(job, max(1, args.steps // 2))
        line["kv_held"] = job.rows_held_curve()
        line["kept_sets"] = job.kept_set_curve()
        line["prefill_attend"] = prefill_attend_leg(wl, device)
        if wl.name == "llava15_7b":   # and the longest prompt of the workloads (LLaVA-NeXT shape, 8 sequences x 32 heads)
            line["prefill_attend_long_prompt"] = prefill_attend_leg(get_workload("llava_next_b8"), device, max_instances=256)
            torch.cuda.empty_cache()
        # the oracle on the host cores, bounded sample
        ns = 96 if wl.batch == 1 else max(1, 96 // wl.batch)    # about 10-20 s of host time
        K, V, q0 = job.K.cpu(), job.V.cpu(), job.q0.cpu()
        q, kn, vn = job.q[:ns + 2].cpu(), job.kn[:ns + 2].cpu(), job.vn[:ns + 2].cpu()
        val, secs, threads, s_first, s_last = oracle_sample(wl, job.g, K, V, q0, q, kn, vn, ns, 2)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "threads": f"numpy fp64; the Python loop over (layer, sequence) is serial, the "
                                           f"matrix products inside it use a BLAS pool of {threads} thread(s)",
                                "sample": f"all {wl.num_layers} layers x {wl.batch} sequence(s), decode steps "
                                          f"{s_first}-{s_last} of {wl.decode_steps} after the oracle's own prefill "
                                          f"({secs:.1f} s)"}
        # the other LLaVA-shaped workloads, one generation each
        if wl.name == "llava15_7b" and not args.no_others:
            job.ctx.close()
            del job
            torch.cuda.empty_cache()
            line["all_workloads"] = [other_workload_line(n, device, local)
                                     for n in ("llava15_7b_b32", "llava15_13b_b16", "llava_next_b8")]
            job = None
        # oracle and GPU free-running side by side (no re-seeding): where, if anywhere, the kept sets part
        line["free_running"] = free_running_report(wl, device)
    if rank == 0:
        print(json.dumps(line))
    if job is not None:
        job.ctx.close()
    if dist:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
