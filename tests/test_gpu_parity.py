"""Parity of the CUDA path (through the C ABI) against the fp64 oracle on the synthetic workloads."""
import numpy as np
import pytest
import torch

from synth import SynthInputs, get_workload
from gpu_harness import run_and_check, GpuRun

pytestmark = pytest.mark.gpu


def test_generator_is_bit_identical_on_cpu_and_gpu():
    wl = get_workload("llava15_7b")
    g = SynthInputs(wl)
    Kc, Vc = g.kv_rows([0], [7], range(0, wl.t0_max, 3))
    Kg, Vg = g.kv_rows([0], [7], range(0, wl.t0_max, 3), device="cuda:0")
    assert torch.equal(Kc, Kg.cpu()) and torch.equal(Vc, Vg.cpu())
    assert torch.equal(g.queries([0, 5], [7]), g.queries([0, 5], [7], device="cuda:0").cpu())


@pytest.mark.parametrize("tau,overlap", [(50.0, False), (10.0, False), (50.0, True)])
def test_tiny_every_step(tau, overlap):
    wl = get_workload("tiny").scaled(tau=tau)
    stats = run_and_check(wl, wl.decode_steps, overlap=overlap)
    assert stats["units"] == wl.decode_steps + 1


@pytest.mark.parametrize("rows", [16, 64, 100, 128])
def test_tiny_chunk_sizes_and_ragged_tails(rows):
    wl = get_workload("tiny")
    run_and_check(wl, 6, rows_per_chunk=rows)


def test_tiny_untrimmed_equals_full_attention():
    wl = get_workload("tiny")
    stats = run_and_check(wl, 4, disable_trim=1)
    assert stats["near-tie"] == 0


@pytest.mark.parametrize("dtype,D,H", [("f32", 128, 3), ("bf16", 64, 5), ("bf16", 128, 2), ("f32", 64, 1)])
def test_small_odd_shapes(dtype, D, H):
    wl = get_workload("tiny").scaled(dtype=dtype, head_dim=D, num_heads=H, num_layers=5, batch=3, sys_len=3,
                                     num_visual=131, text_len_min=1, text_len_max=37, decode_steps=9,
                                     first_prune_layer=1, stride=2, step_ratio_bp=2000, tau=9.0, num_planted=7)
    run_and_check(wl, 9)
    run_and_check(wl, 5, layers_per_call=2)
    run_and_check(wl, 9, layers_per_call=2, overlap=True)


def test_largest_visual_span_and_head_count():
    """Close to the largest visual span the library accepts (8192; the seeded generator numbers at most 8192
    tokens per sequence, prompt and generated) for the top-k and the compaction, and the generator's largest
    head count, on otherwise small shapes."""
    wl = get_workload("tiny").scaled(dtype="bf16", head_dim=64, num_heads=2, num_layers=2, batch=2, sys_len=5,
                                     num_visual=8150, text_len_min=3, text_len_max=20, decode_steps=4,
                                     first_prune_layer=0, stride=1, step_ratio_bp=1500, tau=6.0, num_planted=200)
    run_and_check(wl, 4)
    wl = get_workload("tiny").scaled(dtype="bf16", head_dim=128, num_heads=64, num_layers=2, batch=1, sys_len=4,
                                     num_visual=96, text_len_min=9, text_len_max=9, decode_steps=3,
                                     first_prune_layer=0, stride=1, step_ratio_bp=2500, tau=5.0, num_planted=9)
    run_and_check(wl, 3)


def test_no_visual_tokens_and_single_text_token():
    wl = get_workload("tiny").scaled(num_visual=0, num_planted=0, sys_len=0, text_len_min=1, text_len_max=1,
                                     decode_steps=3)
    run_and_check(wl, 3)


def test_llava15_7b_first_steps_all_units():
    wl = get_workload("llava15_7b")
    stats = run_and_check(wl, 3)
    assert stats["units"] == 32 * 4


@pytest.mark.parametrize("overlap", [False, True])
def test_llava15_7b_full_length_sampled_steps(overlap):
    """`overlap`: consecutive steps overlap on the GPU (the mode bench.py times) or run in plain stream order."""
    wl = get_workload("llava15_7b")
    steps = [0, 1, 2, 17, 64, 128, 129, 200, 254, 255, 256]
    stats = run_and_check(wl, wl.decode_steps, check_steps=steps, overlap=overlap)
    assert stats["units"] == 32 * len(steps)


def _sampled_units(wl, n, seed):
    r = np.random.default_rng(seed)
    layers = [0, 3, wl.num_layers - 1] + r.integers(0, wl.num_layers, size=n).tolist()
    return [(int(r.integers(wl.batch)), int(l)) for l in layers]


def _covering_units(wl, n, seed):
    """At least n distinct (sequence, layer) units: every pruning layer (stage head), the first and the last
    layer, the sequences with the shortest and the longest text, the rest drawn at random."""
    r = np.random.default_rng(seed)
    text = SynthInputs(wl).text_len
    b_short, b_long = int(np.argmin(text)), int(np.argmax(text))
    heads = list(range(wl.first_prune_layer, wl.num_layers, wl.stride))
    units = {(b_short, 0), (b_long, wl.num_layers - 1), (b_long, 1), (b_short, wl.num_layers - 1)}
    for i, l in enumerate(heads):
        units.add(((b_short, b_long)[i % 2], l))
        units.add((int(r.integers(wl.batch)), l))
    while len(units) < n:
        units.add((int(r.integers(wl.batch)), int(r.integers(wl.num_layers))))
    return sorted(units, key=lambda u: (u[1], u[0]))


@pytest.mark.parametrize("name,steps", [("llava15_7b_b32", [0, 1, 100, 300, 511, 512]),
                                        ("llava15_13b_b16", [0, 1, 256, 511, 512]),
                                        ("llava_next_b8", [0, 1, 500, 1023, 1024])])
def test_full_size_workloads_sampled_units(name, steps):
    """The batched workloads at full size and full length, launched as bench.py launches them (all layers per
    call, steps overlapping): 32 or more units, every pruning layer among them, are judged at the sampled steps."""
    wl = get_workload(name)
    units = _covering_units(wl, 32, wl.seed)
    assert len(units) >= 32
    stats = run_and_check(wl, wl.decode_steps, check_steps=steps, units=units, rows_checks=2, overlap=True)
    assert stats["units"] == len(units) * len(steps)


def test_static_rank_mode_tiny_and_small():
    """Algorithm 3 as printed: kept rows in top-index order, decode cuts a prefix before attending."""
    wl = get_workload("tiny")
    stats = run_and_check(wl, wl.decode_steps, static_rank=1)
    assert stats["units"] == wl.decode_steps + 1
    wl = get_workload("tiny").scaled(dtype="bf16", head_dim=128, num_heads=3, num_layers=5, batch=2, sys_len=3,
                                     num_visual=131, text_len_min=1, text_len_max=37, decode_steps=9,
                                     first_prune_layer=1, stride=2, step_ratio_bp=2000, tau=9.0, num_planted=7)
    run_and_check(wl, 9, static_rank=1)


def test_static_rank_mode_llava15_7b():
    wl = get_workload("llava15_7b")
    steps = [0, 1, 2, 100, 255, 256]
    stats = run_and_check(wl, wl.decode_steps, check_steps=steps, static_rank=1)
    assert stats["units"] == 32 * len(steps)


@pytest.mark.parametrize("static_rank", [0, 1])
def test_prefill_with_external_scores_then_decode(static_rank):
    """Algorithm 1's order: prune by scores from outside (the previous layer's alpha), then attend."""
    wl = get_workload("tiny").scaled(dtype="bf16", head_dim=128, num_heads=4, num_layers=6, batch=3, sys_len=4,
                                     num_visual=300, text_len_min=2, text_len_max=30, decode_steps=8,
                                     first_prune_layer=2, stride=2, step_ratio_bp=1500, tau=8.0, num_planted=9)
    run = GpuRun(wl, static_rank=static_rank)
    try:
        g = torch.Generator().manual_seed(7)
        scores = torch.randn(wl.num_layers, wl.batch, wl.num_visual, generator=g).cuda()     # negatives included
        scores[1, 0, 5] = scores[1, 0, 17]                                                   # an exact tie
        run.prefill_scored(scores)
        for l in range(wl.num_layers):
            for b in range(wl.batch):
                run.check_prefill_scored_unit(b, l, scores)
                run.check_rows_unit(b, l, (l + b) % wl.num_heads, 0)
        for t in range(1, 5):                                    # decode goes on from the externally chosen set
            before = run.snapshot(range(wl.num_layers))
            run.decode(t)
            for l in range(wl.num_layers):
                for b in range(wl.batch):
                    run.check_decode_unit(b, l, t, before[l])
        assert run.ctx.status() == 0
    finally:
        run.close()


@pytest.mark.parametrize("static_rank,lpc", [(0, None), (1, None), (0, 1), (0, 3)])
def test_stage_shared_sets(static_rank, lpc):
    """Layers between two pruning layers keep exactly the pruning layer's tokens (strided pruning)."""
    wl = get_workload("tiny").scaled(dtype="bf16", head_dim=128, num_heads=4, num_layers=9, batch=2, sys_len=4,
                                     num_visual=260, text_len_min=2, text_len_max=30, decode_steps=10,
                                     first_prune_layer=2, stride=3, step_ratio_bp=1500, tau=10.0, num_planted=9)
    stats = run_and_check(wl, 10, layers_per_call=lpc, stage_shared=1, static_rank=static_rank)
    assert stats["units"] == 11 * 9 * 2


def test_stage_shared_llava15_7b_first_steps():
    wl = get_workload("llava15_7b")
    stats = run_and_check(wl, 3, stage_shared=1)
    assert stats["units"] == 32 * 4


def test_qk_heredity_lazy_layers():
    """Lazy layers attend with their source layer's probabilities and their own values (Eq. 6)."""
    wl = get_workload("tiny").scaled(dtype="bf16", head_dim=128, num_heads=4, num_layers=9, batch=2, sys_len=4,
                                     num_visual=260, text_len_min=2, text_len_max=30, decode_steps=10,
                                     first_prune_layer=2, stride=3, step_ratio_bp=1500, tau=10.0, num_planted=9)
    # stages: [2,3,4] [5,6,7] [8]; lazy: 1 (source 0, unpruned), 3 and 4 (source 2), 7 (source 6)
    lazy = (1 << 1) | (1 << 3) | (1 << 4) | (1 << 7)
    stats = run_and_check(wl, 10, stage_shared=1, lazy_mask=lazy)
    assert stats["units"] == 11 * 9 * 2


@pytest.mark.parametrize("dtype,head_dim,overlap", [("bf16", 128, True), ("f32", 64, False), ("f32", 128, True),
                                                    ("bf16", 64, False)])
def test_qk_heredity_runs_of_lazy_layers(dtype, head_dim, overlap):
    """Runs of lazy layers of odd and even length (their value rows follow their source's work item through its
    ring slot two layers at a time), below the first pruning layer and inside a pruning stage; every kernel
    instantiation; cache rows of lazy layers (values appended, no keys stored) compared bit for bit."""
    wl = get_workload("tiny").scaled(dtype=dtype, head_dim=head_dim, num_heads=3, num_layers=12, batch=2, sys_len=3,
                                     num_visual=150, text_len_min=1, text_len_max=70, decode_steps=8,
                                     first_prune_layer=7, stride=5, step_ratio_bp=1000, tau=9.0, num_planted=7)
    lazy = sum(1 << l for l in (1, 2, 3, 4, 5, 8, 9, 10, 11))     # 0 -> 1..5, 6 on its own, 7 -> 8..11
    stats = run_and_check(wl, 8, stage_shared=1, lazy_mask=lazy, overlap=overlap,
                          rows_units=[(0, 0), (1, 3), (0, 4), (1, 5), (0, 7), (1, 9), (0, 11)])
    assert stats["units"] == 9 * 12 * 2


def test_qk_heredity_configuration_errors():
    from paper_2412_20105_b200 import binding as B
    wl = get_workload("tiny").scaled(num_layers=9, first_prune_layer=2, stride=3, step_ratio_bp=1500)
    for kw in (dict(lazy_mask=1), dict(lazy_mask=1 << 3), dict(lazy_mask=1 << 5, stage_shared=1),
               dict(lazy_mask=1 << 2, stage_shared=1), dict(lazy_mask=1 << 9, stage_shared=1)):
        with pytest.raises(B.St3Error):
            B.st3_workspace_size(B.config_from_workload(wl, **kw))
    B.st3_workspace_size(B.config_from_workload(wl, lazy_mask=(1 << 3) | (1 << 4), stage_shared=1))


def test_paper_style_configuration_on_llava15_7b():
    """7B schedule with shared stages and the paper's lazy pattern inside the last full stage
    (layers 29 and 30 inherit layer 28; layer 31 starts a new stage and cannot be lazy)."""
    wl = get_workload("llava15_7b")
    lazy = (1 << 29) | (1 << 30)
    steps = [0, 1, 2, 60, 255, 256]
    stats = run_and_check(wl, wl.decode_steps, check_steps=steps, stage_shared=1, lazy_mask=lazy)
    assert stats["units"] == 32 * len(steps)


def test_stage_shared_13b_sampled():
    wl = get_workload("llava15_13b_b16")
    units = _sampled_units(wl, 6, 11) + [(0, 3), (0, 4), (0, 6), (5, 7), (5, 8)]
    units = sorted(set(units), key=lambda u: (u[1], u[0]))
    # a follower is judged against its pruning layer: make sure every sampled follower has it in the list
    heads = sorted(set((b, 3 + (l - 3) // 4 * 4) for b, l in units if l >= 3))
    units = sorted(set(units) | set(heads), key=lambda u: (u[1], u[0]))
    stats = run_and_check(wl, 40, check_steps=[0, 1, 20, 40], units=units, rows_checks=1, stage_shared=1)
    assert stats["units"] == len(units) * 4


@pytest.mark.parametrize("name", ["tiny", "llava15_7b"])
def test_free_running_against_the_oracle(name):
    """Oracle and GPU run a whole generation without either adopting the other's state.  Where the kept sets
    part (if they do) the oracle's scores at that cut must be a near-tie; until then outputs stay in tolerance."""
    import bench
    from gpu_harness import OUT_ABS_F32, OUT_REL_BF16
    wl = get_workload(name)
    rep = bench.free_running_report(wl, torch.device("cuda:0"))
    print("free-running:", rep)
    assert rep["steps_compared"] == wl.decode_steps and rep["units"] == wl.num_layers * wl.batch
    first = rep["first_divergence"]
    assert first is None or first["near_tie"], first
    if first is None:
        assert rep["units_diverged_by_the_end"] == 0
    assert rep["max_output_error_while_in_agreement"] <= (OUT_ABS_F32 if wl.dtype == "f32" else OUT_REL_BF16)
