"""Pins for the oracle's prefill-end selection (window scores, pooling, top-k,
compaction).  CPU only."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.ndimage import maximum_filter1d

from oracle import catekv_oracle as orc
from workloads import synth
from test_oracle_attention import _golden


def test_window_scores_against_library_softmax():
    rng = np.random.default_rng(10)
    G, L_obs, n, d = 3, 5, 40, 16
    qw = orc.f64_to_bf16(rng.standard_normal((G, L_obs, d)))
    k = orc.f64_to_bf16(rng.standard_normal((n, d)))
    C = orc.window_scores(qw, k, L_obs)
    assert C.shape == (n - L_obs,)
    Q = torch.from_numpy(orc.bf16_to_f64(qw))
    K = torch.from_numpy(orc.bf16_to_f64(k))[: n - L_obs]
    A = torch.softmax(torch.einsum("gid,jd->gij", Q, K) / math.sqrt(d), dim=-1)
    np.testing.assert_allclose(C, A.sum(dim=1).mean(dim=0).numpy(), rtol=1e-12)
    # every softmax row sums to one -> C sums to L_obs whatever the data
    assert abs(C.sum() - L_obs) < 1e-12


def test_window_scores_closed_form_identical_keys():
    # all scored keys equal -> uniform rows -> C_j = L_obs / (n - L_obs)
    G, L_obs, n, d = 2, 4, 20, 8
    rng = np.random.default_rng(11)
    qw = orc.f64_to_bf16(rng.standard_normal((G, L_obs, d)))
    k = np.tile(orc.f64_to_bf16(rng.standard_normal((1, d))), (n, 1))
    k[n - L_obs:] = orc.f64_to_bf16(rng.standard_normal((L_obs, d)))  # window keys are not scored
    C = orc.window_scores(qw, k, L_obs)
    np.testing.assert_allclose(C, np.full(n - L_obs, L_obs / (n - L_obs)), rtol=1e-14)


def test_pooling_against_library_routines():
    rng = np.random.default_rng(12)
    C = rng.random(53)
    S, cand_end = 3, 47
    np.testing.assert_array_equal(orc.pool_scores(C, S, cand_end, orc.POOL_NONE, 0), C[S:cand_end])
    for w in (1, 3, 7, 9):
        want = maximum_filter1d(C, size=w, mode="constant", cval=-np.inf)[S:cand_end]
        np.testing.assert_array_equal(orc.pool_scores(C, S, cand_end, orc.POOL_SLIDING, w), want)
    for cs in (1, 4, 8):
        ncand = cand_end - S
        nfull = ncand // cs
        want = C[S:S + nfull * cs].reshape(nfull, cs).max(axis=1)
        got = orc.pool_scores(C, S, cand_end, orc.POOL_CHUNK, cs)
        np.testing.assert_array_equal(got[:nfull], want)
        if ncand % cs:
            assert got.shape[0] == nfull + 1 and got[-1] == C[S + nfull * cs:cand_end].max()


def test_select_hand_example(golden_dir):
    g = _golden(golden_dir, "hand_examples.txt")
    l = [0.0, math.log(2), math.log(4), math.log(2), 0.0, 0.0]
    # d = 2 is not a bf16-friendly size for ln 2; use the float path of the oracle directly
    K = np.array([[x, 0.0] for x in l])
    Q = np.array([[1.0, 0.0]])
    A = orc._row_softmax((Q @ K[:5].T) / 1.0)  # scale 1 in the example
    C = A.sum(axis=0)
    want_C = [float(Fraction(x)) for x in g["select_C"]]
    np.testing.assert_allclose(C, want_C, rtol=1e-15)
    kept = [int(x) for x in g["select_kept"]]
    # the tie between tokens 1 and 3 must be exact for the tie-break to be exercised
    Cx = np.array(want_C)
    assert Cx[1] == Cx[3]
    for mode, param in ((orc.POOL_NONE, 0), (orc.POOL_SLIDING, 3), (orc.POOL_CHUNK, 2)):
        idx = orc.select_indices(Cx, 6, 1, 1, 4, mode, param)
        assert list(idx) == kept, (mode, list(idx))


def test_select_hand_example_through_bf16_inputs():
    # the same example with bf16-exact logits 0, 1, 2, 1, 0, 0 and scale folded into d = 1
    k = orc.f64_to_bf16(np.array([[0.0], [1.0], [2.0], [1.0], [0.0], [0.0]]))
    qw = orc.f64_to_bf16(np.array([[[1.0]]]))
    C = orc.window_scores(qw, k, 1)
    e = math.e
    Z = 2 + 2 * e + e * e
    np.testing.assert_allclose(C, np.array([1, e, e * e, e, 1]) / Z, rtol=1e-14)
    idx = orc.select_indices(C, 6, 1, 1, 4, orc.POOL_NONE, 0)
    assert list(idx) == [0, 1, 2, 5]


def _brute_force_topk(P, k):
    """Best k-subset by total score; among equal totals the lexicographically
    smallest index tuple.  Exponential: tiny inputs only."""
    best, best_sum = None, None
    for comb in itertools.combinations(range(len(P)), k):
        s = math.fsum(P[i] for i in comb)
        if best is None or s > best_sum:  # combinations come in lexicographic order
            best, best_sum = comb, s
    return list(best) if best is not None else []


def test_select_brute_force_subsets():
    rng = np.random.default_rng(13)
    for trial in range(30):
        n = int(rng.integers(8, 15))
        S, Lc = int(rng.integers(0, 3)), int(rng.integers(1, 3))
        T = int(rng.integers(S + Lc, n))
        # dyadic scores: subset sums are exact, ties are exact
        C = rng.integers(0, 6, size=n - 1).astype(np.float64) / 8.0
        idx = orc.select_indices(C, n, S, Lc, T, orc.POOL_NONE, 0)
        k_rest = T - S - Lc
        cand = list(range(S, n - Lc))
        sel = _brute_force_topk([C[j] for j in cand], k_rest)
        want = list(range(S)) + [cand[i] for i in sel] + list(range(n - Lc, n))
        assert list(idx) == want, (trial, list(idx), want)
        assert len(idx) == min(n, T)


def test_select_brute_force_chunks():
    """CHUNK mode against subset enumeration: the best floor(k_rest / cs) chunks by total BlockMax, ties to the
    lexicographically smallest chunk tuple; chunk origin at S, short last chunk included."""
    rng = np.random.default_rng(16)
    short_last = 0
    for trial in range(40):
        cs = int(rng.choice([2, 3]))
        n = int(rng.integers(12, 24))
        S, Lc = int(rng.integers(0, 4)), int(rng.integers(1, 4))
        T = int(rng.integers(S + Lc, n))
        C = rng.integers(0, 7, size=n - 1).astype(np.float64) / 8.0  # dyadic: exact sums, exact ties
        cand_end = n - Lc
        chunks = [list(range(lo, min(lo + cs, cand_end))) for lo in range(S, cand_end, cs)]
        short_last += len(chunks[-1]) < cs
        block_max = [max(C[j] for j in ch) for ch in chunks]  # BlockMax written out, not through pool_scores
        n_take = (T - S - Lc) // cs
        sel = _brute_force_topk(block_max, n_take)
        want = list(range(S)) + [j for c in sel for j in chunks[c]] + list(range(cand_end, n))
        idx = orc.select_indices(C, n, S, Lc, T, orc.POOL_CHUNK, cs)
        assert list(idx) == want, (trial, cs, list(idx), want)
    assert short_last >= 5  # the ragged last chunk was exercised


def test_select_structure_and_modes_agree():
    rng = np.random.default_rng(14)
    n, S, Lc, T = 500, 4, 32, 100
    C = rng.random(n - 32)
    a = orc.select_indices(C, n, S, Lc, T, orc.POOL_NONE, 0)
    b = orc.select_indices(C, n, S, Lc, T, orc.POOL_SLIDING, 1)
    c = orc.select_indices(C, n, S, Lc, T, orc.POOL_CHUNK, 1)
    assert np.array_equal(a, b) and np.array_equal(a, c)
    for idx in (a, orc.select_indices(C, n, S, Lc, T, orc.POOL_SLIDING, 7),
                orc.select_indices(C, n, S, Lc, T, orc.POOL_CHUNK, 8)):
        assert np.all(np.diff(idx) > 0)
        assert list(idx[:S]) == list(range(S))
        assert list(idx[-Lc:]) == list(range(n - Lc, n))
    assert len(a) == T
    # chunks: floor(k_rest / cs) whole chunks
    d = orc.select_indices(C, n, S, Lc, T, orc.POOL_CHUNK, 8)
    assert len(d) == S + Lc + ((T - S - Lc) // 8) * 8
    mid = d[S:-Lc]
    assert np.all((mid - S) % 8 == np.tile(np.arange(8), len(mid) // 8))
    # the top-k of NONE are exactly the k_rest largest candidate scores
    thr = np.sort(C[S:n - Lc])[::-1][T - S - Lc - 1]
    assert np.all(C[a[S:-Lc]] >= thr)
    # budget at or above n, or sink + local covering the sequence: keep everything
    assert np.array_equal(orc.select_indices(C, n, S, Lc, n, orc.POOL_NONE, 0), np.arange(n))
    assert np.array_equal(orc.select_indices(C[:4], 36, S, 32, 10, orc.POOL_NONE, 0), np.arange(36))
    # zero top-k slots: sink and local only
    e = orc.select_indices(C, n, S, Lc, S + Lc, orc.POOL_SLIDING, 7)
    assert list(e) == list(range(S)) + list(range(n - Lc, n))


def test_tie_break_lowest_index():
    C = np.array([0.0, 0.5, 0.5, 0.5, 0.5, 0.25, 0.0, 0.0])
    idx = orc.select_indices(C, 9, 1, 1, 4, orc.POOL_NONE, 0)
    assert list(idx) == [0, 1, 2, 8]
    # sliding max replicates maxima: ties are the norm there
    C2 = np.array([0.0, 0.0, 0.9, 0.0, 0.0, 0.0, 0.8, 0.0, 0.0])
    idx = orc.select_indices(C2, 10, 0, 1, 3, orc.POOL_SLIDING, 3)
    assert list(idx) == [1, 2, 9]


def test_planted_keys_are_selected_and_cache_rows_match():
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=1024, budget=68 + 16)  # k_rest = 16 = the planted keys
    p = synth.prefill_layer(w, 0)
    qw, k, v = synth.bits(p["q_win"]), synth.bits(p["k"]), synth.bits(p["v"])
    mask = p["head_mask"]
    cache, idx = orc.select_compact(qw, k, v, p["seq_len"], mask, w.budget, 1.0, w.sink, w.local, w.L_obs,
                                    orc.POOL_NONE, 0)
    for h in range(w.Hkv):
        i = idx[h]
        if mask[0, h]:
            assert len(i) == w.budget
            assert set(p["heavy"][0, h]) <= set(i.tolist())
        else:
            assert np.array_equal(i, np.arange(w.n))
        assert np.array_equal(cache.k_rows[h], k[0, h][i])
        assert np.array_equal(cache.v_rows[h], v[0, h][i])


def test_kept_fraction_matches_paper(golden_dir):
    with open(f"{golden_dir}/kept_fraction.txt") as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for kind, r, eta, budget, n, pct, tol in rows:
        budget, n, pct, tol = int(budget), int(n), float(pct), float(tol)
        if kind == "budget_share":
            got = 100.0 * orc.kept_fraction(0.0, 1.0, budget, n)
        else:
            got = 100.0 * orc.kept_fraction(float(r), float(eta), budget, n)
        assert abs(got - pct) <= tol, (kind, got, pct)
    # the same accounting from actual kept lists
    n, S, Lc = 4096, 4, 64
    C = np.random.default_rng(15).random(n - 32)
    lens = [len(orc.select_indices(C, n, S, Lc, orc.token_budget(n, cons, 256, 1.0), orc.POOL_NONE, 0))
            for cons in (1, 1, 1, 0, 0)]
    assert sum(lens) / (5 * n) == pytest.approx(orc.kept_fraction(0.4, 1.0, 256, n))
    assert orc.token_budget(1000, False, 64, 0.9) == 900
    assert orc.token_budget(1001, False, 64, 0.9) == 900


def test_streaming_head_keeps_sink_and_recent_only():
    # third head type (Section 4.2.4): budget = sink + local, no top-k slot
    assert orc.token_budget(5000, orc.HEAD_STREAMING, 256, 0.9, 4, 64) == 68
    assert orc.token_budget(5000, orc.HEAD_CONSISTENT, 256, 0.9, 4, 64) == 256
    assert orc.token_budget(5000, orc.HEAD_ADAPTIVE, 256, 0.9, 4, 64) == 4500
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=600, Hq=12, Hkv=3)
    p = synth.prefill_layer(w, 0)
    mask = np.array([[2, 1, 0]], dtype=np.uint8)
    cache, idx = orc.select_compact(synth.bits(p["q_win"]), synth.bits(p["k"]), synth.bits(p["v"]), p["seq_len"], mask,
                                    128, 1.0, w.sink, w.local, w.L_obs, orc.POOL_NONE, 0)
    assert list(idx[0]) == list(range(4)) + list(range(600 - 64, 600))
    assert len(idx[1]) == 128 and len(idx[2]) == 600


def test_attention_recall_pins(golden_dir):
    # hand example: full weights [1,2,4,2,1,1]/11, kept {0,1,2,5} -> 8/11
    l = [0.0, math.log(2), math.log(4), math.log(2), 0.0, 0.0]
    K = np.array([[x, 0.0] for x in l])
    q = np.array([1.0, 0.0])
    g = _golden(golden_dir, "hand_examples.txt")
    assert orc.attention_recall(q, K, [0, 1, 2, 5], 1.0) == pytest.approx(float(Fraction(g["recall_kept"][0])), rel=1e-14)
    assert orc.attention_recall(q, K, list(range(6)), 1.0) == pytest.approx(1.0, rel=1e-14)
    # identical keys: recall = |kept| / n
    K2 = np.tile(np.array([[0.3, -0.7]]), (10, 1))
    assert orc.attention_recall(q, K2, [1, 5, 9], 1.0) == pytest.approx(0.3, rel=1e-14)
    # recall = exp(lse_kept - lse_full), the identity the device path uses; and additivity over disjoint sets
    rng = np.random.default_rng(50)
    K3, q3 = rng.standard_normal((200, 16)), rng.standard_normal(16)
    kept = np.sort(rng.choice(200, 40, replace=False))
    rest = np.setdiff1d(np.arange(200), kept)
    _, lse_k = orc.attention(q3, K3[kept], K3[kept], 0.25)
    _, lse_f = orc.attention(q3, K3, K3, 0.25)
    r = orc.attention_recall(q3, K3, kept, 0.25)
    assert r == pytest.approx(math.exp(lse_k - lse_f), rel=1e-12)
    assert r + orc.attention_recall(q3, K3, rest, 0.25) == pytest.approx(1.0, rel=1e-12)
    # brute force with Python floats
    s = [0.25 * sum(float(a) * float(b) for a, b in zip(K3[j], q3)) for j in range(200)]
    Z = math.fsum(math.exp(x) for x in s)
    assert r == pytest.approx(math.fsum(math.exp(s[j]) for j in kept) / Z, rel=1e-12)


def test_window_attention_against_library_sdpa_and_brute_force():
    rng = np.random.default_rng(60)
    G, L_obs, n, d = 3, 5, 23, 16
    qw = orc.f64_to_bf16(rng.standard_normal((G, L_obs, d)))
    k = orc.f64_to_bf16(rng.standard_normal((n, d)))
    v = orc.f64_to_bf16(rng.standard_normal((n, d)))
    out, lse = orc.window_attention(qw, k, v, L_obs)
    Q = torch.from_numpy(orc.bf16_to_f64(qw))
    K = torch.from_numpy(orc.bf16_to_f64(k))
    V = torch.from_numpy(orc.bf16_to_f64(v))
    pos = torch.arange(n - L_obs, n)[:, None]
    allowed = torch.arange(n)[None, :] <= pos                      # [L_obs, n]: causal prefix of every window row
    ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None, None].expand(1, G, n, d),
                                                           V[None, None].expand(1, G, n, d), attn_mask=allowed)[0]
    np.testing.assert_allclose(out, ref.numpy(), rtol=1e-12, atol=1e-14)
    logits = torch.einsum("gid,jd->gij", Q, K) / math.sqrt(d)
    ref_lse = torch.logsumexp(logits.masked_fill(~allowed, -math.inf), dim=-1)
    np.testing.assert_allclose(lse, ref_lse.numpy(), rtol=1e-13)
    # pure Python, one row: the last window row sees every key, the first one n - L_obs + 1 keys
    for g, i in ((0, L_obs - 1), (2, 0)):
        q = [float(x) for x in orc.bf16_to_f64(qw[g, i])]
        m = n - L_obs + i + 1
        s = [sum(a * float(b) for a, b in zip(q, orc.bf16_to_f64(k[j]))) / math.sqrt(d) for j in range(m)]
        Z = math.fsum(math.exp(x) for x in s)
        want = [math.fsum(math.exp(s[j]) * float(orc.bf16_to_f64(v[j])[e]) for j in range(m)) / Z for e in range(d)]
        np.testing.assert_allclose(out[g, i], want, rtol=1e-12)
        assert lse[g, i] == pytest.approx(math.log(Z), rel=1e-13)


def test_window_attention_closed_form_identical_keys():
    # identical keys: uniform weights over the causal prefix -> the mean of its values, lse = logit + log(prefix)
    rng = np.random.default_rng(61)
    G, L_obs, n, d = 2, 4, 12, 8
    qw = orc.f64_to_bf16(rng.standard_normal((G, L_obs, d)))
    k = np.tile(orc.f64_to_bf16(rng.standard_normal((1, d))), (n, 1))
    v = orc.f64_to_bf16(rng.standard_normal((n, d)))
    out, lse = orc.window_attention(qw, k, v, L_obs)
    V = orc.bf16_to_f64(v)
    for g in range(G):
        for i in range(L_obs):
            m = n - L_obs + i + 1
            np.testing.assert_allclose(out[g, i], V[:m].mean(axis=0), rtol=1e-13, atol=1e-15)
            logit = float(orc.bf16_to_f64(qw[g, i]) @ orc.bf16_to_f64(k[0])) / math.sqrt(d)
            assert lse[g, i] == pytest.approx(logit + math.log(m), rel=1e-13)


def test_criticality_from_the_prefill_log_sum_exp():
    # the scored range's normaliser against a library logsumexp, its relation to the causal one, and C rebuilt from it
    rng = np.random.default_rng(62)
    G, L_obs, n, d = 4, 6, 50, 16
    qw = orc.f64_to_bf16(rng.standard_normal((G, L_obs, d)))
    k = orc.f64_to_bf16(rng.standard_normal((n, d)))
    v = orc.f64_to_bf16(rng.standard_normal((n, d)))
    _, lse_full = orc.window_attention(qw, k, v, L_obs)
    lse_sel = orc.scored_range_lse(qw, k, L_obs)
    Q = torch.from_numpy(orc.bf16_to_f64(qw))
    K = torch.from_numpy(orc.bf16_to_f64(k))
    logits = torch.einsum("gid,jd->gij", Q, K) / math.sqrt(d)
    np.testing.assert_allclose(lse_sel, torch.logsumexp(logits[:, :, : n - L_obs], dim=-1).numpy(), rtol=1e-13)
    # exp(lse_full) = exp(lse_scored) + the window's own causal keys
    for g in range(G):
        for i in range(L_obs):
            own = math.fsum(math.exp(float(logits[g, i, j])) for j in range(n - L_obs, n - L_obs + i + 1))
            assert math.exp(lse_full[g, i]) == pytest.approx(math.exp(lse_sel[g, i]) + own, rel=1e-12)
    C = orc.window_scores_from_lse(qw, k, L_obs, lse_sel)
    np.testing.assert_allclose(C, orc.window_scores(qw, k, L_obs), rtol=1e-11)
    assert abs(C.sum() - L_obs) < 1e-10
