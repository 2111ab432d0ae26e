"""The workspace-free attention entry point against the regular one.

`st3_attend_noalloc` serves callers that are not allowed to allocate device memory (a plugin that
only receives its input and output tensors, code inside a memory region some other allocator owns,
a process with no device memory to spare): its split partials live in a fixed array inside the
library instead of a caller-provided workspace.  Here it must reproduce what `st3_prefill_select`
computes for the same prompt (one layer, one sequence, text rows only), on two calls in a row, the
second smaller than the first so that the shared array still holds the first call's partials.

This file is named to be collected last.
"""
import pytest
import torch

from paper_2412_20105_b200 import binding as B
from paper_2412_20105_b200.build import build
from gpu_harness import assert_out_close
from helpers import f64

pytestmark = pytest.mark.gpu


def _regular(q, k, v, dtype):
    """out[h] via the workspace-based entry point: a prompt of T text rows, nothing visual."""
    H, T, D = k.shape
    cfg = B.make_config(num_layers=1, num_heads=H, head_dim=D, dtype=dtype, batch=1, sys_len=0, num_visual=0,
                        max_text_len=T, max_decode_steps=0, stride=1, step_ratio_bp=0, tau=1.0)
    ctx = B.Context(cfg)
    out = torch.empty((1, 1, H, D), dtype=q.dtype, device=q.device)
    ctx.prefill_select(q.view(1, 1, H, D), k.view(1, 1, H, T, D), v.view(1, 1, H, T, D), [T], out)
    assert ctx.status() == 0
    res = out[0, 0].clone()
    ctx.close()
    return res


def _inputs(seed, H, T, D, dtype):
    g = torch.Generator(device="cpu").manual_seed(seed)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    mk = lambda *s: torch.randn(*s, generator=g).to(tdt).cuda()
    return mk(H, D) * 2.0, mk(H, T, D), mk(H, T, D)


# every kernel instance (element type x head size), with row counts that make one chunk, a chunk boundary, a
# ragged last chunk of a single row, and a single-row input
CASES = [(32, 675, 128, "bf16"), (8, 200, 64, "f32"), (5, 129, 64, "bf16"), (3, 127, 128, "f32"),
         (4, 1, 128, "f32"), (2, 1, 64, "bf16"), (7, 128, 64, "bf16"), (6, 257, 128, "bf16")]


def _check_call(seed, H, T, D, dtype, stream):
    q, k, v = _inputs(seed, H, T, D, dtype)
    out = torch.empty_like(q)
    B.st3_attend_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), H, T, D, dtype, stream)
    torch.cuda.synchronize()
    ref = _regular(q, k, v, dtype)
    assert_out_close(f64(out), f64(ref), dtype, f"noalloc call {seed}")
    # and both agree with plain softmax attention in fp64
    p = torch.softmax(torch.einsum("htd,hd->ht", k.double(), q.double()) / D ** 0.5, dim=1)
    assert_out_close(f64(out), f64(torch.einsum("ht,htd->hd", p, v.double())), dtype, f"noalloc vs fp64 {seed}")


def test_two_calls_in_a_row_match_the_workspace_path():
    build()
    stream = torch.cuda.current_stream().cuda_stream
    for seed, (H, T, D, dtype) in enumerate(CASES[:2]):
        _check_call(seed, H, T, D, dtype, stream)


@pytest.mark.parametrize("first,second", [(0, 2), (2, 3), (3, 4), (1, 5), (6, 7), (7, 0)])
def test_every_kernel_instance_and_ragged_row_counts(first, second):
    """Two calls in a row again, over all four (element type, head size) instances and the chunk edge cases;
    the second call runs on whatever partials the first one left in the shared array."""
    build()
    stream = torch.cuda.current_stream().cuda_stream
    for i in (first, second):
        _check_call(100 + i, *CASES[i], stream)


def test_sizes_beyond_the_static_array_are_rejected():
    build()
    q = torch.zeros(128, 128, device="cuda")
    with pytest.raises(B.St3Error) as e:
        # 128 heads x 65 chunks of 128 rows = 8320 partial slots > 8192; pointers are never dereferenced
        B.st3_attend_noalloc(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), 128, 65 * 128, 128, "f32", 0)
    assert e.value.code == 4
