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


def test_pruning_layers_chained_over_kept_tokens():
    """Algorithm 1 over three pruning layers back to back: the causal attention of layer l runs on the tokens
    layer l kept ([S | kept V | I], in sequence order), its last row gives alpha^l by ORIGINAL visual index
    (st3_prefill_attend_kept), and that prunes layer l+1 before it attends (st3_prefill_select_scored, Eq. 3).
    The oracle walks the same chain with causal_attention and prefill_select_scored; every kept set is judged
    with the near-tie rule on the oracle's scores and is nested in the previous layer's."""
    from helpers import check_kept
    build()
    L, H, sys_len, nv, text = 3, 3, 5, 150, 21
    T = sys_len + nv + text
    g = torch.Generator().manual_seed(11)
    mk = lambda *shape: torch.randn(*shape, generator=g).to(torch.bfloat16).cuda()
    Q, K, V = mk(L, H, T, 128), mk(L, H, T, 128), mk(L, H, T, 128)       # the full prompt of every layer
    Qp, Kp, Vp = mk(H, T, 128), mk(H, T, 128), mk(H, T, 128)             # the layer ahead of the first pruning layer
    # keys of a few visual tokens pulled toward the last query so that the scores have structure
    for t in (Kp, K[0], K[1], K[2]):
        t[:, sys_len + 7:sys_len + nv:9] += 0.25 * (Qp[:, -1:] if t is Kp else Q[0, :, -1:])
    cfg = B.make_config(num_layers=L, num_heads=H, head_dim=128, dtype="bf16", batch=1, sys_len=sys_len, num_visual=nv,
                        max_text_len=text, max_decode_steps=2, stride=1, step_ratio_bp=1500, first_prune_layer=0,
                        tau=4.0)
    st = torch.cuda.current_stream().cuda_stream
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    f64 = lambda t: t.double().cpu().numpy()

    def attend_kept(q, k, v, ids_sorted):
        """GPU: causal attention over [S | ids_sorted | I] of one layer's prompt -> (out, scores by original id)."""
        n = len(ids_sorted)
        rows = torch.tensor(list(range(sys_len)) + [sys_len + int(i) for i in ids_sorted] +
                            list(range(sys_len + nv, T)), device="cuda")
        qs, ks, vs = (t.index_select(1, rows).contiguous() for t in (q, k, v))
        out = torch.empty_like(qs)
        probs = torch.zeros(H, max(1, n), device="cuda")
        scores = torch.full((1, nv), 7.0, device="cuda")
        ids_dev = torch.tensor(ids_sorted, dtype=torch.int32, device="cuda").reshape(1, -1)
        B.st3_prefill_attend_kept(qs.data_ptr(), ks.data_ptr(), vs.data_ptr(), out.data_ptr(), probs.data_ptr(),
                                  scores.data_ptr(), status.data_ptr(), H, H, len(rows), 128, "bf16", sys_len, n,
                                  ids_dev.data_ptr(), nv, st)
        ref_out, A = O.causal_attention(f64(qs), f64(ks), f64(vs))
        bound = 2.0 ** -8 * (np.matmul(A, np.abs(f64(vs))) + np.abs(ref_out)) + 1e-6
        assert (np.abs(f64(out) - ref_out) - bound).max() <= 0
        ref_scores = np.full(nv, -1.0)
        ref_scores[np.asarray(ids_sorted, dtype=np.int64)] = A[:, -1, sys_len:sys_len + n].sum(axis=0)
        return scores, ref_scores

    ctx = B.Context(cfg)
    try:
        scores, ref_scores = attend_kept(Qp, Kp, Vp, list(range(nv)))       # alpha of the layer ahead: all tokens
        held = set(range(nv))
        out = torch.empty(1, 1, H, 128, dtype=torch.bfloat16, device="cuda")
        for l in range(L):
            got = scores[0].cpu().numpy()
            mask = ref_scores >= 0
            assert np.array_equal(got[~mask], ref_scores[~mask])            # tokens not held: exactly -1
            assert np.allclose(got[mask], ref_scores[mask], rtol=2e-3, atol=1e-7)
            n_l = B.st3_schedule_count(cfg, l, 0)
            ctx.prefill_select_scored(Q[l, :, -1].reshape(1, 1, H, 128).contiguous(), K[l].reshape(1, 1, H, T, 128),
                                      V[l].reshape(1, 1, H, T, 128), [text], scores.reshape(1, 1, nv), out,
                                      layer_begin=l)
            ids, cnt, _ = ctx.get_kept(l)
            kept = ids[0, :int(cnt[0])].cpu().numpy()
            assert check_kept(ref_scores, np.arange(nv), n_l, kept) in ("exact", "near-tie")
            assert set(kept.tolist()) <= held and len(kept) == n_l
            held = set(kept.tolist())
            # the layer's output for the last prompt token, on the rows it kept (oracle on the GPU's kept set)
            forced = np.where(np.isin(np.arange(nv), kept), 1.0, 0.0)
            ref_o, _ = O.prefill_select_scored(f64(Q[l, :, -1]), f64(K[l]), f64(V[l]), sys_len, nv, n_l, forced)
            rel = np.abs(f64(out[0, 0]) - ref_o) / np.maximum(np.abs(ref_o), 1e-2)
            assert rel.max() <= 2e-2
            scores, ref_scores = attend_kept(Q[l], K[l], V[l], sorted(held))  # alpha^l prunes layer l+1
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and ctx.status() == 0
    finally:
        ctx.close()


def test_unsupported_shapes_are_refused():
    x = torch.zeros(1, 8, 64, device="cuda")
    with pytest.raises(B.St3Error) as e:
        B.st3_prefill_attend(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), None, None, None, 1, 1, 8, 64,
                             "bf16", 0, 0, 0)
    assert e.value.code == 7
