"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and its
schedule and argument validation behave (no GPU work)."""
import ctypes as C
import os
import re

import pytest

from oracle.st3_oracle import Schedule
from paper_2412_20105_b200 import binding as B
from paper_2412_20105_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build()


def _cfg(**kw):
    base = dict(num_layers=32, num_heads=32, head_dim=128, dtype="bf16", batch=1, sys_len=35, num_visual=576,
                max_text_len=64, max_decode_steps=256, stride=7, step_ratio_bp=1225, tau=256)
    base.update(kw)
    return B.make_config(**base)


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "st3.h")).read()
    declared = set(re.findall(r"\b(st3_[a-z_]+)\s*\(", hdr))
    assert declared == set(B.EXPORTS)
    lib = B.load()
    for name in declared:
        assert hasattr(lib, name), name


def test_config_struct_matches_header_order():
    hdr = open(os.path.join(ROOT, "include", "st3.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} st3_config;", hdr, re.S).group(1)
    fields = re.findall(r"(?:int32_t|uint64_t|double)\s+([a-z_]+);", body)
    assert fields == [f[0] for f in B.Config._fields_]


@pytest.mark.parametrize("kw", [
    dict(), dict(num_layers=40, num_heads=40, stride=4, step_ratio_bp=500, tau=512, max_decode_steps=512),
    dict(num_visual=2880, tau=1024, max_decode_steps=1024), dict(tau=50), dict(tau=10),
    dict(anneal=B.ST3_ANNEAL_LINEAR, tau=50), dict(anneal=B.ST3_ANNEAL_EXP, sigma=20.0),
    dict(anneal=B.ST3_ANNEAL_NONE), dict(disable_trim=1), dict(first_prune_layer=0, stride=1, step_ratio_bp=175),
])
def test_schedule_matches_oracle(kw):
    cfg = _cfg(**kw)
    an = {0: "cosine", 1: "none", 2: "linear", 3: "exp"}[cfg.anneal]
    s = Schedule(num_layers=cfg.num_layers, num_visual=cfg.num_visual, stride=cfg.stride,
                 step_ratio_bp=cfg.step_ratio_bp, tau=cfg.tau, first_ratio_bp=cfg.first_ratio_bp,
                 first_prune_layer=cfg.first_prune_layer, anneal=an, sigma=cfg.sigma,
                 disable_trim=bool(cfg.disable_trim))
    for l in range(cfg.num_layers):
        for t in range(cfg.max_decode_steps + 1):
            assert B.st3_schedule_count(cfg, l, t) == s.n(l, t), (l, t)


def test_argument_validation_without_gpu():
    assert B.st3_schedule_count(_cfg(), 32, 0) == -1
    assert B.st3_schedule_count(_cfg(head_dim=96), 0, 0) == -1
    with pytest.raises(B.St3Error):
        B.st3_workspace_size(_cfg(num_layers=0))
    with pytest.raises(B.St3Error):
        B.st3_workspace_size(_cfg(rows_per_chunk=1000))
    n = B.st3_workspace_size(_cfg())
    assert n > 32 * 32 * (576 + 35 + 64 + 256) * 128 * 2 * 2        # at least the K/V cache itself
    lib = B.load()
    h = C.c_void_p(None)
    assert lib.st3_create(C.byref(_cfg()), None, n, C.byref(h)) == 1 and h.value is None
    assert lib.st3_create(C.byref(_cfg()), 4096 + 8, n, C.byref(h)) == 1      # misaligned workspace
    assert lib.st3_create(C.byref(_cfg()), 4096, 16, C.byref(h)) == 2         # too small, checked before any CUDA call
    assert lib.st3_decode_step(None, 1, 0, 1, None, None, None, None, None) == 1
    assert lib.st3_destroy(None) == 1
    assert B.st3_status_string(3) == "call order violated"


def test_workspace_grows_by_the_prompt_staging_areas_only_on_request():
    """host_prefill = 1 adds two slots of one layer's prompt K and V (each rounded up to 256 bytes), nothing else."""
    a = B.st3_workspace_size(_cfg())
    b = B.st3_workspace_size(_cfg(host_prefill=1))
    layer = 1 * 32 * (35 + 576 + 64) * 128 * 2                     # B * H * t0_max * D * bytes
    assert b - a == 2 * 2 * ((layer + 255) // 256 * 256)
    # the decode staging (two slots of q | k_new | v_new and of out) is always there: the size depends on L, B, H, D
    assert B.st3_workspace_size(_cfg(num_layers=16)) < a


def test_host_buffer_calls_validate_before_touching_the_gpu():
    lib = B.load()
    assert lib.st3_prefill_select_host(None, 0, 1, None, None, None, None, None, None) == 1
    assert lib.st3_decode_step_host(None, 1, 0, 1, None, None, None, None, None) == 1
    assert lib.st3_host_sync(None, None) == 1
    assert lib.st3_prefill_attend_kept(None, None, None, None, None, None, None, 1, 1, 8, 128, 1, 0, 0, None, 8,
                                       None) == 1
