"""Causal prompt attention on the tensor cores (st3_prefill_attend) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import st3_oracle as O
from paper_2412_20105_b200 import binding as B
from paper_2412_20105_b200.build import build

pytestmark = pytest.mark.gpu


def _run(T, H, nb, sys_len, nv, seed, poison=None):
    build()
    g = torch.Generator().manual_seed(seed)
    n = nb * H
    mk = lambda: torch.randn(n, T, 128, generator=g).to(torch.bfloat16).cuda()
    q, k, v = mk(), mk(), mk()
    if poison is not None:
        poison(q, k, v)
    out = torch.full((n, T, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    probs = torch.zeros(n, max(1, nv), device="cuda")
    scores = torch.zeros(nb, max(1, nv), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.st3_prefill_attend(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), probs.data_ptr(), scores.data_ptr(),
                         status.data_ptr(), n, H, T, 128, "bf16", sys_len, nv, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return q, k, v, out, scores


@pytest.mark.parametrize("T,H,nb,sys_len,nv", [(128, 2, 1, 8, 64), (37, 1, 2, 3, 20), (300, 3, 2, 10, 200),
                                               (675, 4, 1, 35, 576)])
def test_causal_attention_and_next_layer_scores(T, H, nb, sys_len, nv):
    q, k, v, out, scores = _run(T, H, nb, sys_len, nv, seed=T)
    for b in range(nb):
        sl = slice(b * H, (b + 1) * H)
        ref, A = O.causal_attention(q[sl].double().cpu().numpy(), k[sl].double().cpu().numpy(),
                                    v[sl].double().cpu().numpy())
        got = out[sl].double().cpu().numpy()
        # The probabilities enter the second MMA as bf16 (8 significant bits), the output is bf16 too:
        # |err| <= 2^-9 sum_j A_ij |V_jd| (rounding of P) + 2^-9 |ref| (rounding of out); twice that is allowed.
        bound = 2.0 ** -8 * (np.matmul(A, np.abs(v[sl].double().cpu().numpy())) + np.abs(ref)) + 1e-6
        assert np.all(np.isfinite(got))
        excess = np.abs(got - ref) - bound
        assert excess.max() <= 0, f"causal out b={b}: error exceeds the bf16 bound by {excess.max()}"
        want = A[:, T - 1, sys_len:sys_len + nv].sum(axis=0)            # alpha: last row, visual slice, over heads
        assert np.allclose(scores[b, :nv].cpu().numpy(), want, rtol=2e-3, atol=1e-7)


@pytest.mark.parametrize("T", [37, 100, 131])
def test_tiles_never_read_the_neighbouring_instance(T):
    """T is not a multiple of the 64-key tile: the last key tile of an instance reaches past its end.  The rows
    it would find there in a flat layout are the NEXT instance's first rows; they hold Inf/NaN here.  Keys past
    the end carry probability 0, and 0 x Inf = NaN would poison the output if those rows were ever loaded; rows
    outside the instance must read as zeros instead."""
    H, nb, sys_len, nv = 2, 2, 3, 20

    def poison(q, k, v):
        # the first rows of every instance but the first (what the previous instance's last tile overhangs)
        v[1:, :64] = float("inf")
        k[1:, :64] = float("nan")
        q[1:, :64] = float("nan")

    q, k, v, out, scores = _run(T, H, nb, sys_len, nv, seed=T, poison=poison)
    ref, A = O.causal_attention(q[:1].double().cpu().numpy(), k[:1].double().cpu().numpy(), v[:1].double().cpu().numpy())
    got = out[0].double().cpu().numpy()                  # instance 0 is clean; its neighbour is poisoned
    assert np.all(np.isfinite(got))
    bound = 2.0 ** -8 * (np.matmul(A, np.abs(v[:1].double().cpu().numpy())) + np.abs(ref)) + 1e-6
    assert (np.abs(got - ref[0]) - bound[0]).max() <= 0


def test_full_prompt_length_sampled_rows():
    """LLaVA-NeXT prompt length (35 + 2880 + 128), two sequences of 32 heads: a grid of several waves with two
    blocks per SM, as bench.py launches it.  Sampled query rows (tile edges, first, last, a ragged tail) are
    checked one by one against the oracle's single-query attention over the causal prefix; the next layer's
    scores of both sequences against the oracle's last row."""
    T, H, nb, sys_len, nv = 3043, 32, 2, 35, 2880
    q, k, v, out, scores = _run(T, H, nb, sys_len, nv, seed=11)
    rows = [0, 1, 63, 64, 127, 128, 129, 1471, 1472, 2943, 2944, 3007, 3041, 3042]
    for inst in (0, 21, 40, 63):
        K = k[inst:inst + 1].double().cpu().numpy()
        V = v[inst:inst + 1].double().cpu().numpy()
        for r in rows:
            ref, pr = O.attend(q[inst:inst + 1, r].double().cpu().numpy(), K[:, :r + 1], V[:, :r + 1])
            got = out[inst, r].double().cpu().numpy()
            bound = 2.0 ** -8 * (pr[0] @ np.abs(V[0, :r + 1]) + np.abs(ref[0])) + 1e-6
            assert np.all(np.isfinite(got))
            assert (np.abs(got - ref[0]) - bound).max() <= 0, f"instance {inst} row {r}"
    for b in range(nb):
        sl = slice(b * H, (b + 1) * H)
        _, pr = O.attend(q[sl, T - 1].double().cpu().numpy(), k[sl].double().cpu().numpy(), v[sl].double().cpu().numpy())
        want = O.visual_mass(pr, sys_len, nv)
        assert np.allclose(scores[b, :nv].cpu().numpy(), want, rtol=2e-3, atol=1e-7)


def test_scores_feed_the_scored_prefill():
    """The scores of one layer's causal attention prune the next layer's prompt (Eq. 3's alpha^{l-1})."""
    T, H, sys_len, nv, text = 96, 2, 4, 80, 12
    q, k, v, out, scores = _run(T, H, 1, sys_len, nv, seed=5)
    cfg = B.make_config(num_layers=1, num_heads=H, head_dim=128, dtype="bf16", batch=1, sys_len=sys_len, num_visual=nv,
                        max_text_len=text, max_decode_steps=2, stride=1, step_ratio_bp=0, first_prune_layer=0,
                        tau=4.0)
    ctx = B.Context(cfg)
    try:
        o2 = torch.empty(1, 1, H, 128, dtype=torch.bfloat16, device="cuda")
        ctx.prefill_select_scored(q[:, -1].reshape(1, 1, H, 128).contiguous(), k.reshape(1, 1, H, T, 128),
                                  v.reshape(1, 1, H, T, 128), [text], scores[:, :nv].reshape(1, 1, nv).contiguous(), o2)
        ids, cnt, _ = ctx.get_kept(0)
        n = int(cnt[0])
        assert n == nv // 2
        top = np.argsort(-scores[0, :nv].cpu().numpy(), kind="stable")[:n]
        assert sorted(ids[0, :n].tolist()) == sorted(top.tolist())
        assert ctx.status() == 0
    finally:
        ctx.close()


def test_unsupported_shapes_are_refused():
    x = torch.zeros(1, 8, 64, device="cuda")
    with pytest.raises(B.St3Error) as e:
        B.st3_prefill_attend(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), None, None, None, 1, 1, 8, 64,
                             "bf16", 0, 0, 0)
    assert e.value.code == 7
