"""Pins for the oracle's query-aware retrieval (chunk min/max upper bound, chunk top-k).  CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import catekv_oracle as orc
from workloads import synth


def test_metadata_is_elementwise_extremes():
    rng = np.random.default_rng(60)
    k = orc.f64_to_bf16(rng.standard_normal((21, 6)))
    kmax, kmin = orc.retrieval_metadata(k, 8)
    K = orc.bf16_to_f64(k)
    assert kmax.shape == (3, 6)
    for c, (lo, hi) in enumerate([(0, 8), (8, 16), (16, 21)]):
        for e in range(6):
            assert kmax[c, e] == max(K[t, e] for t in range(lo, hi))
            assert kmin[c, e] == min(K[t, e] for t in range(lo, hi))
    # chunk size 1: both are the row itself
    a, b = orc.retrieval_metadata(k, 1)
    assert np.array_equal(a, K) and np.array_equal(b, K)


def test_scores_bound_every_row_and_are_tight_for_single_rows():
    rng = np.random.default_rng(61)
    K = rng.standard_normal((64, 16))
    k = orc.f64_to_bf16(K)
    Kb = orc.bf16_to_f64(k)
    q = rng.standard_normal((3, 16))
    kmax, kmin = orc.retrieval_metadata(k, 8)
    s = orc.retrieval_scores(q, kmax, kmin)
    logits = q @ Kb.T  # [G, rows]
    for c in range(8):
        # the defining property: no row of the chunk can score above the chunk's bound, for any head of the group
        assert s[c] >= logits[:, c * 8:(c + 1) * 8].max() - 1e-12
    # pure-Python evaluation of the bound
    for c in (0, 5):
        best = -math.inf
        for g in range(3):
            tot = math.fsum(max(float(q[g, e]) * float(kmin[c, e]), float(q[g, e]) * float(kmax[c, e])) for e in range(16))
            best = max(best, tot)
        assert s[c] == pytest.approx(best, rel=1e-13)
    # chunk size 1: the bound is the exact best logit of the group
    a, b = orc.retrieval_metadata(k, 1)
    np.testing.assert_allclose(orc.retrieval_scores(q, a, b), logits.max(axis=0), rtol=1e-13, atol=1e-13)
    # sign split used by the device path: max(q kmin, q kmax) = max(q,0) kmax + min(q,0) kmin
    alt = np.maximum(q, 0) @ kmax.T + np.minimum(q, 0) @ kmin.T
    np.testing.assert_allclose(s, alt.max(axis=0), rtol=1e-13, atol=1e-13)


def _brute(P, k):
    best, bs = None, None
    for comb in itertools.combinations(range(len(P)), k):
        t = math.fsum(P[i] for i in comb)
        if best is None or t > bs:
            best, bs = comb, t
    return list(best) if best else []


def test_retrieve_indices_brute_force_and_structure():
    rng = np.random.default_rng(62)
    for trial in range(20):
        cs = int(rng.choice([1, 2, 4]))
        n = int(rng.integers(14, 26))
        S, Lc = int(rng.integers(0, 4)), int(rng.integers(1, 6))
        budget = int(rng.integers(S + Lc, n))
        nch = (n + cs - 1) // cs
        scores = rng.integers(0, 5, size=nch).astype(np.float64) / 4.0
        idx = orc.retrieve_indices(scores, n, S, Lc, budget, cs)
        assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] == n - 1
        S2 = (S + cs - 1) // cs * cs
        cand_end = (n - Lc) // cs * cs
        if cand_end <= S2 or (budget - S2 - (n - cand_end)) // cs >= (cand_end - S2) // cs:
            assert np.array_equal(idx, np.arange(n))
            continue
        k_sel = max(0, (budget - S2 - (n - cand_end)) // cs)
        pool = [scores[S2 // cs + c] for c in range((cand_end - S2) // cs)]
        if math.comb(len(pool), k_sel) > 20000:
            continue
        sel = _brute(pool, k_sel)
        want = list(range(S2)) + [S2 + c * cs + e for c in sel for e in range(cs)] + list(range(cand_end, n))
        assert list(idx) == want, (trial, list(idx), want)
        assert len(idx) <= max(budget, S2 + n - cand_end)
        assert set(range(S)) <= set(idx.tolist()) and set(range(n - Lc, n)) <= set(idx.tolist())
    # ties go to the lowest chunk
    sc = np.array([0.0, 1.0, 1.0, 1.0, 1.0, 0.0])
    assert list(orc.retrieve_indices(sc, 24, 4, 4, 16, 4)) == list(range(0, 4)) + list(range(4, 12)) + list(range(20, 24))
    # a budget covering the list keeps every row
    assert np.array_equal(orc.retrieve_indices(sc, 24, 4, 4, 24, 4), np.arange(24))


def test_retrieval_finds_planted_keys_when_the_bound_is_informative():
    # quiet keys (small norm) with a few loud ones along a direction the queries lean on: the chunk bound then
    # separates the loud chunks, they must all be retrieved and carry almost all of the attention mass.
    # (On i.i.d. N(0,1) keys the min/max bound is dominated by noise; that is a property of the criterion.)
    rng = np.random.default_rng(63)
    n, d, G = 2048, 32, 4
    c = rng.standard_normal(d)
    c /= np.linalg.norm(c)
    K = 0.05 * rng.standard_normal((n, d))
    heavy = np.sort(rng.choice(np.arange(16, n - 80), 12, replace=False))
    K[heavy] += 3.0 * c
    k = orc.f64_to_bf16(K)
    Q = 0.1 * rng.standard_normal((G, d)) + 3.0 * c
    kmax, kmin = orc.retrieval_metadata(k, 8)
    s = orc.retrieval_scores(Q, kmax, kmin)
    idx = orc.retrieve_indices(s, n, 4, 64, 256, 8)
    assert len(idx) == 8 + (n - (n - 64) // 8 * 8) + ((256 - 8 - (n - (n - 64) // 8 * 8)) // 8) * 8
    assert set(heavy.tolist()) <= set(idx.tolist())
    rec = [orc.attention_recall(Q[g], orc.bf16_to_f64(k), idx, 1.0) for g in range(G)]
    assert min(rec) > 0.9
