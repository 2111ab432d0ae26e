"""Plain fp64 CPU oracle for ST^3 decode-step attention over a trimmed visual KV cache.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It shares no code with the CUDA path and is not
tuned for speed.  Every function restates a passage of the paper (ST^3,
"Spatial-Temporal Visual Token Trimming") step by step in numpy float64.

Readings taken where the paper is silent or inconsistent (each one is a
documented choice, not a derivation):
  * PVTP ratios are additive in the ORIGINAL visual-token count: the first
    pruning layer removes P, each later pruning layer removes a further R.
    This is the reading that reproduces every (L, S, R) -> C row the paper
    prints in its stride/ratio ablation tables.
  * Pruning layers are l = first, first+S, first+2S, ... (first = 3); the
    layers between two pruning layers keep the count of their stage.
  * VTA count is |V^{l,0}| * beta^t (Eq. 7, non-compounding), floor'ed; with
    |O^t| = t at decode step t (t = 1 consumes the first generated token).
  * The score of a visual token is the sum over heads of the current query's
    attention probability on it (Eq. 2's last row, sliced to visual positions).
  * Top(G, .) breaks equal scores toward the lower original visual index.
  * Attend first, then trim: the cache after step t holds n(l, t) visual rows.
  * Selection at layer l uses layer l's own scores (layer-local trimming).

Pins (tests/test_oracle_*.py): the paper's printed (L, S, R, C) table rows,
closed forms of beta, brute-force softmax in long double, torch SDPA as a
library special case, an O(n^2) exhaustive definition of top-k, and run-long
invariants.  No function here is "parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------
# Retention schedule: PVTP per layer (Sec. 3.2, Eq. 9, Algorithm 1) times
# VTA per decode step (Sec. 3.3, Eq. 7 and Eq. 8).
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Schedule:
    num_layers: int
    num_visual: int
    stride: int                      # S, pruning stride
    step_ratio_bp: int               # R in basis points of num_visual
    tau: float                       # Eq. 8 decay horizon
    first_ratio_bp: int = 5000       # P, "set to 50%" (text under Eq. 9)
    first_prune_layer: int = 3       # layers 0-2 are never pruned (Sec. 3.2)
    anneal: str = "cosine"           # "cosine" | "linear" | "exp" | "none"
    sigma: float = 20.0              # only for anneal == "exp"
    disable_trim: bool = False       # full-KV comparison run

    def stage(self, layer: int) -> int:
        """Index of the pruning stage layer `layer` belongs to (-1: never pruned).

        Algorithm 1 prunes when l >= 3 and (l - 3) % S == 0, so stage heads are
        3, 3+S, 3+2S, ... and every layer up to the next head shares the stage.
        """
        if layer < self.first_prune_layer:
            return -1
        return (layer - self.first_prune_layer) // self.stride

    def keep_bp(self, layer: int) -> int:
        """Fraction of the original visual tokens layer `layer` keeps, in basis points.

        Eq. 9 generalised to every layer: 1 - P - k*R with k the number of
        pruning layers passed after the first one.
        """
        k = self.stage(layer)
        if k < 0 or self.disable_trim:
            return 10000
        return max(0, 10000 - self.first_ratio_bp - k * self.step_ratio_bp)

    def n0(self, layer: int) -> int:
        """|V^{l,0}|: visual tokens kept at layer l after prefill (floor)."""
        return (self.num_visual * self.keep_bp(layer)) // 10000

    def beta(self, t: int) -> float:
        """Eq. 8 (cosine), or the linear / exponential variants of Sec. 4.4."""
        if self.anneal == "none" or self.disable_trim:
            return 1.0
        if self.anneal == "exp":
            return math.exp(-t / self.sigma)
        if t >= self.tau:
            return 0.0
        if self.anneal == "cosine":
            return math.cos(t * math.pi / (2.0 * self.tau))
        if self.anneal == "linear":
            return 1.0 - t / self.tau
        raise ValueError(self.anneal)

    def n(self, layer: int, t: int) -> int:
        """Scheduled visual-row count of layer `layer` after decode step t (Eq. 7)."""
        base = self.n0(layer)
        if layer < self.first_prune_layer or t == 0:
            return base
        return int(math.floor(base * self.beta(t) + 1e-9))


def conserved_fraction_bp(num_layers: int, stride: int, step_ratio_bp: int,
                          first_ratio_bp: int = 5000) -> int:
    """C of Eq. 9 as realised by the schedule: the last layer's keep fraction."""
    s = Schedule(num_layers=num_layers, num_visual=10000, stride=stride,
                 step_ratio_bp=step_ratio_bp, tau=1.0, first_ratio_bp=first_ratio_bp)
    return s.keep_bp(num_layers - 1)


# --------------------------------------------------------------------------
# Attention of the current (last) query, Eq. 2 restricted to its last row.
# --------------------------------------------------------------------------
def attend(q: np.ndarray, K: np.ndarray, V: np.ndarray):
    """Softmax attention of one query per head over all cached rows.

    q [H, D], K [H, T, D], V [H, T, D] (float64).  Returns (out [H, D],
    p [H, T]): p is the last row of A = Softmax((QK^T + M)/sqrt(d)); the last
    row of a causal mask sees every position, itself included.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    d = q.shape[-1]
    logits = np.matmul(K, q[:, :, None])[:, :, 0] / math.sqrt(d)       # [H, T]
    logits = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    p = e / e.sum(axis=1, keepdims=True)
    out = np.matmul(p[:, None, :], V)[:, 0, :]                         # [H, D]
    return out, p


def causal_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray):
    """Eq. 2 in full: A = Softmax((Q K^T + M) / sqrt(d)), out = A V, with M masking the strict upper
    triangle (row i sees keys 0..i).  Q, K, V [H, T, D].  Returns (out [H, T, D], A [H, T, T])."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    T, d = Q.shape[1], Q.shape[2]
    logits = np.matmul(Q, np.swapaxes(K, 1, 2)) / math.sqrt(d)            # [H, T, T]
    mask = np.triu(np.ones((T, T), dtype=bool), k=1)
    logits = np.where(mask[None], -np.inf, logits)
    logits = logits - logits.max(axis=2, keepdims=True)
    e = np.exp(logits)
    A = e / e.sum(axis=2, keepdims=True)
    return np.matmul(A, V), A


def visual_mass(p: np.ndarray, vis_begin: int, n_vis: int) -> np.ndarray:
    """alpha: the query's attention on each visual token, summed over heads."""
    return p[:, vis_begin:vis_begin + n_vis].sum(axis=0)


def select_top(scores: np.ndarray, ids: np.ndarray, k: int) -> np.ndarray:
    """Top(G, alpha) of Eq. 3: positions of the k highest scores.

    Equal scores are ordered by lower original visual index `ids`.  Returns the
    kept positions in ascending position order.
    """
    n = len(scores)
    k = max(0, min(int(k), n))
    order = np.lexsort((np.asarray(ids), -np.asarray(scores, dtype=np.float64)))
    return np.sort(order[:k])


# --------------------------------------------------------------------------
# Per-(sequence, layer) cache state: rows [S | V_kept | I | O_1..O_t].
# --------------------------------------------------------------------------
@dataclass
class LayerCache:
    K_sys: np.ndarray                 # [H, sys, D]
    V_sys: np.ndarray
    K_vis: np.ndarray                 # [H, n_cur, D]
    V_vis: np.ndarray
    ids: np.ndarray                   # [n_cur] original visual index of each kept row
    K_txt: np.ndarray                 # [H, text + generated, D]
    V_txt: np.ndarray
    last_mass: np.ndarray = field(default_factory=lambda: np.zeros(0))

    @property
    def n_cur(self) -> int:
        return int(self.ids.shape[0])

    def rows(self):
        K = np.concatenate([self.K_sys, self.K_vis, self.K_txt], axis=1)
        V = np.concatenate([self.V_sys, self.V_vis, self.V_txt], axis=1)
        return K, V


def rank_order(scores: np.ndarray, ids: np.ndarray) -> np.ndarray:
    """Positions sorted by descending score, equal scores by lower original index: the saved
    top-index list T[l] of Algorithm 3.  Every prefix of it is a Top(G, .) of Eq. 3."""
    return np.lexsort((np.asarray(ids), -np.asarray(scores, dtype=np.float64)))


def prefill_select(q_last, K, V, sys_len: int, num_visual: int, n_keep: int, rank_ordered: bool = False,
                   select_scores=None):
    """Prefill half of Algorithm 3 for one (sequence, layer).

    K, V [H, T0, D] hold the prompt rows [S | V | I]; q_last [H, D] is the last
    prompt token's query.  Attends over the whole prompt, scores the visual
    tokens, keeps the n_keep best (Eq. 3) and builds the cache.
    With rank_ordered the kept rows are stored in the order of the top-index list (best first),
    which is what the static-rank decode of Algorithm 3 truncates.
    select_scores [num_visual], if given, replaces this layer's own scores in the selection: the
    layers between two pruning layers reuse the pruning layer's choice (Sec. 3.2, strided pruning).
    Returns (out [H, D], mass [num_visual], cache).
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    out, p = attend(q_last, K, V)
    mass = visual_mass(p, sys_len, num_visual)
    sel = mass if select_scores is None else np.asarray(select_scores, dtype=np.float64)
    ids_all = np.arange(num_visual, dtype=np.int64)
    if rank_ordered:
        kept = rank_order(sel, ids_all)[:max(0, min(int(n_keep), num_visual))]
    else:
        kept = select_top(sel, ids_all, n_keep)
    v0, v1 = sys_len, sys_len + num_visual
    cache = LayerCache(
        K_sys=K[:, :v0].copy(), V_sys=V[:, :v0].copy(),
        K_vis=K[:, v0:v1][:, kept].copy(), V_vis=V[:, v0:v1][:, kept].copy(),
        ids=ids_all[kept].copy(),
        K_txt=K[:, v1:].copy(), V_txt=V[:, v1:].copy(),
        last_mass=mass,
    )
    return out, mass, cache


def prefill_select_scored(q_last, K, V, sys_len: int, num_visual: int, n_keep: int, scores,
                          rank_ordered: bool = False):
    """Prefill of one (sequence, layer) the way Algorithm 1 / Eq. 3 word it: the visual tokens are
    pruned BEFORE the layer runs, by scores that come from outside (the previous layer's alpha),
    and the layer then attends over [S | kept V | I] only.
    Returns (out [H, D], cache).
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    scores = np.asarray(scores, dtype=np.float64)
    ids_all = np.arange(num_visual, dtype=np.int64)
    if rank_ordered:
        kept = rank_order(scores, ids_all)[:max(0, min(int(n_keep), num_visual))]
    else:
        kept = select_top(scores, ids_all, n_keep)
    v0, v1 = sys_len, sys_len + num_visual
    cache = LayerCache(
        K_sys=K[:, :v0].copy(), V_sys=V[:, :v0].copy(),
        K_vis=K[:, v0:v1][:, kept].copy(), V_vis=V[:, v0:v1][:, kept].copy(),
        ids=ids_all[kept].copy(),
        K_txt=K[:, v1:].copy(), V_txt=V[:, v1:].copy(),
        last_mass=scores,
    )
    Kc, Vc = cache.rows()
    out, _ = attend(q_last, Kc, Vc)
    return out, cache


def decode_step(cache: LayerCache, q, k_new, v_new, n_target: int, select_scores=None):
    """Decode half of Algorithm 3 with Eq. 7 for one (sequence, layer), one step.

    Appends the new token's key/value, attends over every cached row, scores
    the current visual rows and, if the schedule asks for fewer rows than are
    held, keeps the n_target best and evicts the rest.
    select_scores (one per visual row held, in cache order), if given, replaces this layer's own
    scores in the selection (a layer that follows its stage's pruning layer).
    Returns (out [H, D], mass over the visual rows held BEFORE the eviction,
    ids held before the eviction).
    """
    k_new = np.asarray(k_new, dtype=np.float64)
    v_new = np.asarray(v_new, dtype=np.float64)
    cache.K_txt = np.concatenate([cache.K_txt, k_new[:, None, :]], axis=1)
    cache.V_txt = np.concatenate([cache.V_txt, v_new[:, None, :]], axis=1)
    K, V = cache.rows()
    out, p = attend(q, K, V)
    n_cur = cache.n_cur
    mass = visual_mass(p, cache.K_sys.shape[1], n_cur)
    ids_before = cache.ids.copy()
    n_new = min(n_cur, int(n_target))
    if n_new < n_cur:
        kept = select_top(mass if select_scores is None else np.asarray(select_scores, dtype=np.float64),
                          cache.ids, n_new)
        cache.K_vis = cache.K_vis[:, kept]
        cache.V_vis = cache.V_vis[:, kept]
        cache.ids = cache.ids[kept]
    cache.last_mass = mass
    return out, mass, ids_before


def decode_step_static(cache: LayerCache, q, k_new, v_new, n_target: int):
    """Decode half of Algorithm 3 as printed, for a cache kept in top-index order.

    T' = T[l][: n] and C = C[T'] come first (the visual rows are cut to the first n_target of the
    saved order, no re-scoring), then the layer attends over what is left plus the new token.
    Returns out [H, D].
    """
    n_new = min(cache.n_cur, int(n_target))
    cache.K_vis = cache.K_vis[:, :n_new]
    cache.V_vis = cache.V_vis[:, :n_new]
    cache.ids = cache.ids[:n_new]
    k_new = np.asarray(k_new, dtype=np.float64)
    v_new = np.asarray(v_new, dtype=np.float64)
    cache.K_txt = np.concatenate([cache.K_txt, k_new[:, None, :]], axis=1)
    cache.V_txt = np.concatenate([cache.V_txt, v_new[:, None, :]], axis=1)
    K, V = cache.rows()
    out, _ = attend(q, K, V)
    return out


def attend_inherited(q_src, K_src, V_own):
    """QK heredity (Eq. 6, Algorithm 2): a lazy layer reuses Softmax(Q^{l-n} (K^{l-n})^T / sqrt(d)) of the
    last non-lazy layer and applies it to its OWN values.  q_src [H, D], K_src [H, T, D] are the source
    layer's query and keys, V_own [H, T, D] the lazy layer's values, row j of both naming the same token."""
    _, p = attend(q_src, K_src, np.zeros_like(np.asarray(V_own, dtype=np.float64)))
    return np.matmul(p[:, None, :], np.asarray(V_own, dtype=np.float64))[:, 0, :]


def decode_step_lazy(cache: LayerCache, cache_src: LayerCache, q_src, v_new, n_target: int, select_scores):
    """One decode step of a lazy layer.  cache_src is the source layer's cache AFTER the source's own
    append of this step and BEFORE its eviction; both caches must hold the same visual tokens in the
    same order (they belong to one pruning stage).  The lazy layer appends only its value row, attends
    with the inherited probabilities and then evicts what its stage's pruning layer evicts.
    Returns out [H, D]."""
    assert np.array_equal(cache.ids, cache_src.ids), "source and lazy layer must hold the same visual rows"
    v_new = np.asarray(v_new, dtype=np.float64)
    cache.V_txt = np.concatenate([cache.V_txt, v_new[:, None, :]], axis=1)
    cache.K_txt = np.concatenate([cache.K_txt, np.zeros_like(v_new)[:, None, :]], axis=1)   # never read
    K_src, _ = cache_src.rows()
    _, V = cache.rows()
    out = attend_inherited(q_src, K_src, V)
    n_cur = cache.n_cur
    n_new = min(n_cur, int(n_target))
    if n_new < n_cur:
        kept = select_top(np.asarray(select_scores, dtype=np.float64), cache.ids, n_new)
        cache.K_vis = cache.K_vis[:, kept]
        cache.V_vis = cache.V_vis[:, kept]
        cache.ids = cache.ids[kept]
    return out


def overlap_n(ids_1, ids_n) -> float:
    """Overlap_n of Eq. 10: |TopK(T_1) ∩ TopK(T_n)| / |TopK(T_1)|, the share of the visual tokens in the first
    decode step's top-K that are in the n-th step's top-K too.  ids_1, ids_n: the two top-K index sets."""
    a = set(int(i) for i in np.asarray(ids_1).ravel())
    b = set(int(i) for i in np.asarray(ids_n).ravel())
    return len(a & b) / len(a) if a else 1.0


def boundary_scores(mass: np.ndarray, ids: np.ndarray, k: int):
    """(s_k, s_{k+1}): the k-th and (k+1)-th scores in selection order (None if absent)."""
    n = len(mass)
    order = np.lexsort((np.asarray(ids), -np.asarray(mass, dtype=np.float64)))
    s_k = float(mass[order[k - 1]]) if 1 <= k <= n else None
    s_k1 = float(mass[order[k]]) if 0 <= k < n else None
    return s_k, s_k1
