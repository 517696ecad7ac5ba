"""CPU oracle for the CateKV hot path (hybrid-head KV-cache attention).

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64 numpy
statement of what the paper defines, written to be checked against the paper by
eye.  It shares no code with the CUDA library and never imports it.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Inputs are bf16 bit patterns (numpy uint16) widened exactly to float64; all
arithmetic is float64.  numpy's matmul / sort / exp are used as steps; nothing
is blocked, fused or reordered beyond what the definitions state.

What each function follows
--------------------------
* observation_matrix, cv_score      : Section 3.2, Eq. 1-4 (GQA mean: last
                                      paragraph of Section 3.2).
* classify_sample, static_head_mask : Eq. 5 and "Reference-Based Static
                                      Identification" (Section 3.2).
* window_scores                     : Algorithm 1, "Calculating token
                                      criticality".
* pool_scores, select_indices       : Algorithm 1, BlockMax / argtopk / Cache().
* HybridCache.append                : the paper is silent; every head's list
                                      grows by the decoded token.
* attention, decode_attention       : Algorithm 1, "Attention(q, k, v)"; the
                                      plain softmax-attention definition.
* window_attention, scored_range_lse, window_scores_from_lse
                                    : Algorithm 1, pre-filling stage: the
                                      attention rows of the last L_obs prefill
                                      queries (what a prefill pass computes for
                                      those positions), their log-sum-exp, and
                                      the token criticality re-derived from it.
* attention_recall                  : Section 3.4 (attention weight recall of a
                                      kept set, Fig. 4).
* token_budget (streaming type)     : Section 4.2.4 (sink + recent heads).
* retrieval_metadata, retrieval_scores, retrieve_indices
                                    : Algorithm 1, decoding stage, "Retrival(q,
                                      cache)" in its query-aware form on adaptive
                                      heads, with the page criterion of Quest that
                                      the paper combines with (Section 4.2.2,
                                      appendix B.2.2; chunk size 8).

Parity pins: every function above is pinned by tests that do not re-use it
(pure-Python brute force, closed forms, hand-worked examples, library
routines).  The paper's accuracy tables are "parity unpinned": they need model
weights and benchmark data and are outside this oracle.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

POOL_NONE = 0
POOL_CHUNK = 1
POOL_SLIDING = 2


# --------------------------------------------------------------------------
# bf16 <-> float64
# --------------------------------------------------------------------------
def bf16_to_f64(bits) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) exactly to float64."""
    u = np.ascontiguousarray(bits).astype(np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16(x) -> np.ndarray:
    """Round float64 to the nearest bf16 (ties to even); returns uint16 bits.

    Works on the value, not through float32, so there is no double rounding:
    x = m * 2**e with 0.5 <= |m| < 1; bf16 keeps 8 significant bits, i.e.
    m is rounded to a multiple of 2**-8.  (bf16 subnormals are not treated
    specially: the hot path's outputs never get near 2**-126.)
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)
    q = np.rint(m * 256.0) / 256.0
    y = np.ldexp(q, e).astype(np.float32)  # exact: y has 8 significant bits
    y = np.where(np.isfinite(x), y, x.astype(np.float32))
    return (np.ascontiguousarray(y).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# Softmax attention (Algorithm 1, decoding stage: output = Attention(q, k, v))
# --------------------------------------------------------------------------
def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> Tuple[np.ndarray, float]:
    """softmax(scale * K q) V for one query vector.

    q [d], K [L, d], V [L, d] float64.  Returns (o [d], lse) with lse the
    natural-log of sum_j exp(scale * q.k_j).  An empty list gives o = 0 and
    lse = -inf.
    """
    L = K.shape[0]
    if L == 0:
        return np.zeros(V.shape[1] if V.ndim == 2 else q.shape[0]), -math.inf
    s = (K @ q) * scale
    m = s.max()
    p = np.exp(s - m)
    l = p.sum()
    o = (p @ V) / l
    return o, float(m + math.log(l))


# --------------------------------------------------------------------------
# Hybrid per-head cache (Section 1 / Section 3.2: a short list for consistent
# heads, most or all of the tokens for adaptive heads)
# --------------------------------------------------------------------------
@dataclass
class HybridCache:
    """Per (sequence, KV head) lists of cached K and V rows, as bf16 bits."""

    B: int
    Hkv: int
    d: int
    k_rows: List[np.ndarray] = field(default_factory=list)  # each [len, d] uint16
    v_rows: List[np.ndarray] = field(default_factory=list)

    def seg(self, b: int, h: int) -> int:
        return b * self.Hkv + h

    def lengths(self) -> np.ndarray:
        return np.array([r.shape[0] for r in self.k_rows], dtype=np.int64)

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """Every head's list gets the new token's (k, v) at its end.

        k_new, v_new: [B, Hkv, d] uint16.  (The paper does not say how decoded
        tokens enter the caches; autoregressive decoding implies they are
        kept, for consistent and adaptive heads alike.)
        """
        for b in range(self.B):
            for h in range(self.Hkv):
                i = self.seg(b, h)
                self.k_rows[i] = np.concatenate([self.k_rows[i], k_new[b, h][None, :]], axis=0)
                self.v_rows[i] = np.concatenate([self.v_rows[i], v_new[b, h][None, :]], axis=0)


def decode_attention(cache: HybridCache, q_bits: np.ndarray, scale: Optional[float] = None,
                     cells: Optional[Sequence[Tuple[int, int]]] = None):
    """Attention of every query head over its KV head's current list.

    q_bits [B, Hq, d] uint16.  Query head hq reads KV head hq // G, G = Hq/Hkv.
    Returns (out [B, Hq, d] float64, lse [B, Hq] float64, natural log).  With
    `cells` (a list of (b, kv_head)) only those groups are computed; the rest
    of `out` is NaN.
    """
    B, Hq, d = q_bits.shape
    G = Hq // cache.Hkv
    if scale is None or scale == 0:
        scale = 1.0 / math.sqrt(d)
    out = np.full((B, Hq, d), np.nan)
    lse = np.full((B, Hq), np.nan)
    todo = cells if cells is not None else [(b, h) for b in range(B) for h in range(cache.Hkv)]
    for (b, h) in todo:
        i = cache.seg(b, h)
        K = bf16_to_f64(cache.k_rows[i])
        V = bf16_to_f64(cache.v_rows[i])
        for g in range(G):
            hq = h * G + g
            o, s = attention(bf16_to_f64(q_bits[b, hq]), K, V, scale)
            out[b, hq] = o
            lse[b, hq] = s
    return out, lse


# --------------------------------------------------------------------------
# Prefill-end selection (Algorithm 1, pre-filling stage)
# --------------------------------------------------------------------------
def _row_softmax(S: np.ndarray) -> np.ndarray:
    m = S.max(axis=1, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    E = np.exp(S - m)
    Z = E.sum(axis=1, keepdims=True)
    return E / np.where(Z > 0, Z, 1.0)


def window_scores(qwin_bits: np.ndarray, k_bits: np.ndarray, L_obs: int) -> np.ndarray:
    """Token criticality C of Algorithm 1 for one KV head.

    qwin_bits [G, L_obs, d]: the last L_obs prefill queries of the G query
    heads that share this KV head.  k_bits [n, d].  For every query head:
    A = softmax(Q_win K[:n-L_obs]^T / sqrt(d)) row-wise over exactly those
    keys, C = sum of A's rows.  The group's C is the mean over its heads
    (Section 3.2, GQA).  Returns C [n - L_obs] float64.
    """
    G, Lw, d = qwin_bits.shape
    assert Lw == L_obs
    n = k_bits.shape[0]
    ns = n - L_obs
    if ns <= 0:
        return np.zeros(0)
    K = bf16_to_f64(k_bits[:ns])
    C = np.zeros(ns)
    for g in range(G):
        Q = bf16_to_f64(qwin_bits[g])
        A = _row_softmax((Q @ K.T) / math.sqrt(d))
        C += A.sum(axis=0)
    return C / G


def window_attention(qwin_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, L_obs: int,
                     scale: Optional[float] = None):
    """The prefill attention of the observation window (Algorithm 1, pre-filling stage: the queries
    Q[-L_obs:] whose scores select the tokens are ordinary prefill queries).

    qwin_bits [G, L_obs, d], k_bits / v_bits [n, d].  Window row i sits at position n - L_obs + i and, being a
    prefill query, attends causally to keys 0 .. n - L_obs + i.  Returns (out [G, L_obs, d], lse [G, L_obs]):
    softmax(scale * q K^T) V over that prefix and the natural-log sum of exp(logits).
    """
    G, Lw, d = qwin_bits.shape
    assert Lw == L_obs
    n = k_bits.shape[0]
    if scale is None or scale == 0:
        scale = 1.0 / math.sqrt(d)
    K, V = bf16_to_f64(k_bits), bf16_to_f64(v_bits)
    out = np.zeros((G, L_obs, d))
    lse = np.zeros((G, L_obs))
    for g in range(G):
        Q = bf16_to_f64(qwin_bits[g])
        for i in range(L_obs):
            pos = n - L_obs + i
            out[g, i], lse[g, i] = attention(Q[i], K[:pos + 1], V[:pos + 1], scale)
    return out, lse


def scored_range_lse(qwin_bits: np.ndarray, k_bits: np.ndarray, L_obs: int) -> np.ndarray:
    """Natural-log sum of exp(q_i . k_j / sqrt(d)) of every window row over the scored keys j < n - L_obs alone:
    the normaliser of the softmax in Algorithm 1's "token criticality" line.  [G, L_obs].
    (It relates to the causal log-sum-exp of window_attention by
    exp(lse_full) = exp(lse_scored) + sum over the window's own keys j <= n - L_obs + i of exp(logit).)"""
    G, Lw, d = qwin_bits.shape
    n = k_bits.shape[0]
    K = bf16_to_f64(k_bits[: n - L_obs])
    out = np.zeros((G, L_obs))
    for g in range(G):
        S = (bf16_to_f64(qwin_bits[g]) @ K.T) / math.sqrt(d)
        m = S.max(axis=1)
        out[g] = m + np.log(np.exp(S - m[:, None]).sum(axis=1))
    return out


def window_scores_from_lse(qwin_bits: np.ndarray, k_bits: np.ndarray, L_obs: int, lse_sel: np.ndarray) -> np.ndarray:
    """Token criticality C of Algorithm 1 with the softmax normaliser given instead of computed:
    C_j = mean_g sum_i exp(q_gi . k_j / sqrt(d) - lse_sel[g, i]) for the scored keys j < n - L_obs."""
    G, Lw, d = qwin_bits.shape
    n = k_bits.shape[0]
    ns = n - L_obs
    K = bf16_to_f64(k_bits[:ns])
    C = np.zeros(ns)
    for g in range(G):
        Q = bf16_to_f64(qwin_bits[g])
        S = (Q @ K.T) / math.sqrt(d)
        C += np.exp(S - lse_sel[g][:, None]).sum(axis=0)
    return C / G


def pool_scores(C: np.ndarray, S: int, cand_end: int, mode: int, param: int) -> np.ndarray:
    """Pooling of the criticality vector before top-k.

    NONE    : P_j = C_j for candidates j in [S, cand_end).
    SLIDING : P_j = max C_t over |t - j| <= (w-1)/2 clipped to the scored range
              (stride-1 max pool, -inf padding), for the same candidates.
    CHUNK   : BlockMax(C, cs) of Algorithm 1: chunk c covers
              [S + c*cs, min(S + (c+1)*cs, cand_end)); P_c = max over the chunk.
    Returns the pooled vector (one entry per candidate token, or per chunk).
    """
    ncand = max(0, cand_end - S)
    if mode == POOL_NONE:
        return C[S:cand_end].copy()
    if mode == POOL_SLIDING:
        w = int(param)
        assert w >= 1 and w % 2 == 1
        half = (w - 1) // 2
        P = np.empty(ncand)
        for idx in range(ncand):
            j = S + idx
            lo = max(0, j - half)
            hi = min(C.shape[0], j + half + 1)
            P[idx] = C[lo:hi].max()
        return P
    if mode == POOL_CHUNK:
        cs = int(param)
        assert cs >= 1
        nch = (ncand + cs - 1) // cs
        P = np.empty(nch)
        for c in range(nch):
            lo = S + c * cs
            hi = min(S + (c + 1) * cs, cand_end)
            P[c] = C[lo:hi].max()
        return P
    raise ValueError("pool mode")


HEAD_ADAPTIVE, HEAD_CONSISTENT, HEAD_STREAMING = 0, 1, 2


def token_budget(n: int, head_type: int, budget_consistent: int, eta_adaptive: float, sink: int = 0,
                 local: int = 0) -> int:
    """T of the head: b for a consistent head (1), floor(eta * n) for an adaptive one (0), and sink + local for a
    streaming head (2: attention sinks and recent tokens only, the head type of the DuoAttention comparison in
    Section 4.2.4)."""
    head_type = int(head_type)
    if head_type == HEAD_STREAMING:
        return int(sink) + int(local)
    if head_type == HEAD_CONSISTENT:
        return int(budget_consistent)
    if eta_adaptive >= 1.0:
        return n
    return int(math.floor(eta_adaptive * n))


def select_indices(C: np.ndarray, n: int, S: int, Lc: int, T: int, mode: int, param: int) -> np.ndarray:
    """Kept token indices of one head, ascending (Algorithm 1: argtopk + Cache()).

    The first S (sink) and last Lc (local) tokens are always kept and count in
    the budget T; the remaining k_rest = max(0, T - S - Lc) slots go to the
    candidates [S, n - Lc) with the largest pooled score, ties to the lowest
    index.  In CHUNK mode floor(k_rest / cs) whole chunks are taken.
    T >= n, or sink and local covering the sequence, keeps everything.
    """
    if T >= n or S + Lc >= n:
        return np.arange(n, dtype=np.int64)
    cand_end = n - Lc
    k_rest = max(0, T - S - Lc)
    P = pool_scores(C, S, cand_end, mode, param)
    # order by (score descending, index ascending): stable sort of -P
    order = np.argsort(-P, kind="stable")
    if mode == POOL_CHUNK:
        cs = int(param)
        take = order[: k_rest // cs]
        sel = []
        for c in take:
            lo = S + int(c) * cs
            hi = min(S + (int(c) + 1) * cs, cand_end)
            sel.extend(range(lo, hi))
        sel = np.array(sorted(sel), dtype=np.int64)
    else:
        sel = np.sort(order[:k_rest]).astype(np.int64) + S
    return np.concatenate([np.arange(S, dtype=np.int64), sel, np.arange(n - Lc, n, dtype=np.int64)])


def select_compact(qwin_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, seq_len: Sequence[int],
                   head_mask: np.ndarray, budget_consistent: int, eta_adaptive: float, S: int, Lc: int,
                   L_obs: int, mode: int, param: int,
                   cells: Optional[Sequence[Tuple[int, int]]] = None):
    """Prefill-end selection and compaction for a batch.

    qwin_bits [B, Hq, L_obs, d]; k_bits, v_bits [B, Hkv, n_max, d]; seq_len[b]
    tokens of sequence b are valid; head_mask [B, Hkv] (1 = consistent).
    Returns (cache, idx) where idx[b*Hkv+h] is the ascending kept index list
    and the cache rows are K/V gathered in that order.  With `cells` only
    those (b, h) are computed; the others get empty lists.
    """
    B, Hq, Lw, d = qwin_bits.shape
    Hkv = k_bits.shape[1]
    G = Hq // Hkv
    assert Lc >= L_obs, "the local window must cover the observation window"
    cache = HybridCache(B, Hkv, d)
    idx_all = []
    want = None if cells is None else set(cells)
    for b in range(B):
        n = int(seq_len[b])
        for h in range(Hkv):
            if want is not None and (b, h) not in want:
                idx = np.zeros(0, dtype=np.int64)
            else:
                T = token_budget(n, int(head_mask[b, h]), budget_consistent, eta_adaptive, S, Lc)
                if T >= n or S + Lc >= n:
                    idx = np.arange(n, dtype=np.int64)
                else:
                    C = window_scores(qwin_bits[b, h * G:(h + 1) * G], k_bits[b, h, :n], L_obs)
                    idx = select_indices(C, n, S, Lc, T, mode, param)
            idx_all.append(idx)
            cache.k_rows.append(k_bits[b, h][idx].copy())
            cache.v_rows.append(v_bits[b, h][idx].copy())
    return cache, idx_all


# --------------------------------------------------------------------------
# Head identification (Section 3.2, Eq. 1-5)
# --------------------------------------------------------------------------
def observation_matrix(qwin_bits: np.ndarray, k_bits: np.ndarray, L_obs: int, L_init: int, L_rec: int,
                       causal: bool) -> np.ndarray:
    """Eq. 1 for one KV head: A [L_obs, m], m = n - L_init - L_rec.

    Per query head: softmax over the sliced keys [L_init, n - L_rec) of
    Q_win K^T / sqrt(d).  With `causal`, window row i (absolute position
    n - L_obs + i) does not see keys after its own position: those entries are
    -inf before the softmax, hence 0 in A.  A is the mean over the group's
    query heads.
    """
    G, Lw, d = qwin_bits.shape
    n = k_bits.shape[0]
    j0, j1 = L_init, n - L_rec
    K = bf16_to_f64(k_bits[j0:j1])
    m = j1 - j0
    A = np.zeros((L_obs, m))
    key_pos = np.arange(j0, j1)[None, :]
    row_pos = (n - L_obs + np.arange(L_obs))[:, None]
    for g in range(G):
        Q = bf16_to_f64(qwin_bits[g])
        Sg = (Q @ K.T) / math.sqrt(d)
        if causal:
            Sg = np.where(key_pos > row_pos, -np.inf, Sg)
        A += _row_softmax(Sg)
    return A / G


def quantile_lower(values: np.ndarray, k: float) -> float:
    """The floor(k * (N-1))-th element of the ascending sort: "the k-th
    percentile element" of Eq. 2, taken as an element of the matrix."""
    flat = np.sort(values.reshape(-1))
    return float(flat[int(math.floor(k * (flat.shape[0] - 1)))])


def cv_from_matrix(A: np.ndarray, quantile_k: float, alpha: float) -> float:
    """Eq. 2-4: binarise at Phi = Quantile_k(A) * alpha (whole matrix), count
    per column, return std_pop(C) / mean(C); a zero mean gives 0."""
    phi = quantile_lower(A, quantile_k) * alpha
    Bm = A >= phi
    C = Bm.sum(axis=0).astype(np.float64)
    mu = C.mean()
    if mu == 0:
        return 0.0
    return float(math.sqrt(((C - mu) ** 2).mean()) / mu)


def cv_score(qwin_bits, k_bits, L_obs, L_init, L_rec, quantile_k, alpha, causal) -> float:
    return cv_from_matrix(observation_matrix(qwin_bits, k_bits, L_obs, L_init, L_rec, causal), quantile_k, alpha)


def head_cv(qwin_bits: np.ndarray, k_bits: np.ndarray, seq_len: Sequence[int], L_obs: int, L_init: int,
            L_rec: int, quantile_k: float, alpha: float, causal: bool) -> np.ndarray:
    """CV score of every (sequence, KV head): [B, Hkv] float64."""
    B, Hq = qwin_bits.shape[:2]
    Hkv = k_bits.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Hkv))
    for b in range(B):
        n = int(seq_len[b])
        for h in range(Hkv):
            out[b, h] = cv_score(qwin_bits[b, h * G:(h + 1) * G], k_bits[b, h, :n], L_obs, L_init, L_rec,
                                 quantile_k, alpha, causal)
    return out


def classify_sample(scores: np.ndarray, r: float) -> np.ndarray:
    """Eq. 5 for one sample: over all heads of the model (flattened), the
    threshold Gamma(r) is the floor(r * (H-1))-th ascending score; a head is
    consistent (1) iff its score is strictly above it."""
    s = np.asarray(scores, dtype=np.float64).reshape(-1)
    gamma = np.sort(s)[int(math.floor(r * (s.shape[0] - 1)))]
    return (s > gamma).astype(np.uint8)


def static_head_mask(cv: np.ndarray, r: float) -> np.ndarray:
    """Reference-based static identification.

    cv [N_samples, H_total].  f_h = number of samples that classify head h as
    consistent (Eq. 5).  n_adapt = floor(r * (H-1)) + 1 heads are adaptive; the
    other H - n_adapt heads, ranked by (f_h descending, mean score descending,
    flat index ascending), are consistent (mask 1).
    """
    cv = np.asarray(cv, dtype=np.float64)
    N, H = cv.shape
    f = np.zeros(H, dtype=np.int64)
    for s in range(N):
        f += classify_sample(cv[s], r)
    mean = cv.mean(axis=0)
    n_adapt = int(math.floor(r * (H - 1))) + 1
    order = sorted(range(H), key=lambda h: (-int(f[h]), -float(mean[h]), h))
    mask = np.zeros(H, dtype=np.uint8)
    for h in order[: H - n_adapt]:
        mask[h] = 1
    return mask


def attention_recall(q: np.ndarray, K: np.ndarray, kept: np.ndarray, scale: float) -> float:
    """Attention recall of a kept set (Section 3.4, the recall curves): the share of the full softmax mass
    of one decode query that falls on the kept tokens, sum_{j in kept} softmax(scale * K q)_j."""
    s = (K @ q) * scale
    p = np.exp(s - s.max())
    p /= p.sum()
    return float(p[np.asarray(kept, dtype=np.int64)].sum())


# --------------------------------------------------------------------------
# Query-aware retrieval on adaptive heads (Algorithm 1: "Retrival(q, cache)")
# --------------------------------------------------------------------------
def retrieval_metadata(k_bits: np.ndarray, cs: int):
    """Per chunk of cs consecutive cached rows: the element-wise maximum and minimum of the keys.
    k_bits [len, d] -> (kmax, kmin), each [ceil(len / cs), d] float64 (values are bf16 values)."""
    K = bf16_to_f64(k_bits)
    L = K.shape[0]
    nch = (L + cs - 1) // cs
    kmax = np.empty((nch, K.shape[1]))
    kmin = np.empty((nch, K.shape[1]))
    for c in range(nch):
        blk = K[c * cs:min((c + 1) * cs, L)]
        kmax[c] = blk.max(axis=0)
        kmin[c] = blk.min(axis=0)
    return kmax, kmin


def retrieval_scores(q_group: np.ndarray, kmax: np.ndarray, kmin: np.ndarray) -> np.ndarray:
    """Upper bound of q.k over the rows of every chunk, per query head sum_d max(q_d kmin_d, q_d kmax_d), and the
    group's score as the maximum over its G query heads.  q_group [G, d] float64 -> [n_chunks]."""
    s = np.full(kmax.shape[0], -np.inf)
    for g in range(q_group.shape[0]):
        q = q_group[g][None, :]
        s = np.maximum(s, np.maximum(q * kmin, q * kmax).sum(axis=1))
    return s


def retrieve_indices(scores: np.ndarray, n: int, S: int, Lc: int, budget: int, cs: int) -> np.ndarray:
    """Rows a retrieval head attends to in one step, ascending.

    Chunks start at row 0.  The chunks that hold the first S rows and every chunk from the one holding row
    n - Lc on are always taken; of the chunks in between, the floor((budget - forced rows) / cs) with the largest
    score, ties to the lowest index.  budget >= n (or no chunk in between) takes every row.
    """
    S2 = (S + cs - 1) // cs * cs                 # sink rows, rounded up to whole chunks
    cand_end = max(0, (n - Lc)) // cs * cs       # first row of the always-taken tail
    if budget >= n or cand_end <= S2:
        return np.arange(n, dtype=np.int64)
    forced = S2 + (n - cand_end)
    n_pool = (cand_end - S2) // cs
    k_sel = max(0, (budget - forced) // cs)
    if k_sel >= n_pool:
        return np.arange(n, dtype=np.int64)
    P = scores[S2 // cs: cand_end // cs]
    order = np.argsort(-P, kind="stable")[:k_sel]
    rows = [np.arange(S2, dtype=np.int64)]
    for c in np.sort(order):
        lo = S2 + int(c) * cs
        rows.append(np.arange(lo, lo + cs, dtype=np.int64))
    rows.append(np.arange(cand_end, n, dtype=np.int64))
    return np.concatenate(rows)


def kept_fraction(r: float, eta: float, budget: int, n: int) -> float:
    """Retained share of the KV cache: adaptive heads (share r) keep eta of the
    tokens, consistent heads keep budget/n (Section 4.2: 2048 of 128K is 1.56 %
    and about 41 % of the cache is retained at r = 0.4, eta = 1)."""
    return r * eta + (1.0 - r) * (budget / n)
