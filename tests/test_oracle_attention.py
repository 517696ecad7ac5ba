"""Pins for the oracle's attention, cache and bf16 helpers (CPU only).

Each test checks the oracle against something that is not the oracle: a library
routine, a closed form, a hand-worked value, a pure-Python brute force, or an
invariant of softmax attention.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import catekv_oracle as orc
from workloads import synth


def _golden(golden_dir, name):
    out = {}
    with open(f"{golden_dir}/{name}") as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = vals
    return out


# ---------------------------------------------------------------- bf16 helpers
def test_bf16_widening_matches_torch():
    u = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    t = torch.from_numpy(u.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = orc.bf16_to_f64(u)
    fin = np.isfinite(t)
    assert np.array_equal(got[fin], t[fin])
    assert np.array_equal(np.isnan(got), np.isnan(t))


def test_bf16_rounding_ties_and_torch():
    # ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even mantissa (1.0)
    assert orc.f64_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    # 1 + 3*2^-8 is halfway between 1 + 2^-7 (odd) and 1 + 2^-6 (even) -> up
    assert orc.f64_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    # just above / below a tie
    assert orc.f64_to_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81
    assert orc.f64_to_bf16(np.array([1.0 + 2.0 ** -8 - 2.0 ** -40]))[0] == 0x3F80
    assert orc.f64_to_bf16(np.array([-2.5]))[0] == 0xC020
    # float32-exact inputs: torch's float32 -> bf16 is round-to-nearest-even
    rng = np.random.default_rng(0)
    x = rng.standard_normal(20000).astype(np.float32)
    want = synth.bits(torch.from_numpy(x).to(torch.bfloat16))
    assert np.array_equal(orc.f64_to_bf16(x.astype(np.float64)), want)
    # round trip of every finite bf16 is the identity
    u = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    v = orc.bf16_to_f64(u)
    ok = np.isfinite(v) & (np.abs(v) >= 2.0 ** -126)
    assert np.array_equal(orc.f64_to_bf16(v[ok]), u[ok])


# ---------------------------------------------------------------- attention
def test_attention_matches_library_sdpa():
    rng = np.random.default_rng(1)
    for L, d in [(1, 8), (7, 16), (64, 128), (300, 128)]:
        q = rng.standard_normal(d)
        K = rng.standard_normal((L, d))
        V = rng.standard_normal((L, d))
        scale = 1.0 / math.sqrt(d)
        o, lse = orc.attention(q, K, V, scale)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[None, None, None, :], torch.from_numpy(K)[None, None],
            torch.from_numpy(V)[None, None], scale=scale)[0, 0, 0].numpy()
        np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)
        ref_lse = torch.logsumexp(torch.from_numpy(K @ q * scale), 0).item()
        assert abs(lse - ref_lse) < 1e-12


def test_attention_pure_python_brute_force_one_head_64_tokens():
    # the 1-head, 64-token brute-force case: Python floats and loops only
    w = synth.scaled(synth.WORKLOADS["cfg0"], Hq=1, Hkv=1, n=64, B=1)
    k = synth.bits(synth.randn_bf16((64, 128), "cpu", 7, "k"))
    v = synth.bits(synth.randn_bf16((64, 128), "cpu", 7, "v"))
    q = synth.bits(synth.randn_bf16((128,), "cpu", 7, "q"))
    K, V, Q = orc.bf16_to_f64(k), orc.bf16_to_f64(v), orc.bf16_to_f64(q)
    scale = 1.0 / math.sqrt(128)
    logits = []
    for j in range(64):
        acc = 0.0
        for e in range(128):
            acc += float(Q[e]) * float(K[j, e])
        logits.append(acc * scale)
    mx = max(logits)
    wts = [math.exp(s - mx) for s in logits]
    Z = math.fsum(wts)
    want = [math.fsum(wts[j] * float(V[j, e]) for j in range(64)) / Z for e in range(128)]
    o, lse = orc.attention(Q, K, V, scale)
    np.testing.assert_allclose(o, np.array(want), rtol=1e-12, atol=1e-14)
    assert abs(lse - (mx + math.log(Z))) < 1e-12
    assert w.G == 1


def test_attention_closed_forms():
    d = 4
    V = np.arange(20, dtype=np.float64).reshape(5, d)
    # identical keys -> uniform weights -> mean of V; lse = s + log L
    K = np.tile(np.array([[0.5, -1.0, 2.0, 0.0]]), (5, 1))
    q = np.array([1.0, 1.0, 1.0, 1.0])
    o, lse = orc.attention(q, K, V, 0.5)
    np.testing.assert_allclose(o, V.mean(axis=0), rtol=1e-15)
    assert abs(lse - (0.75 + math.log(5))) < 1e-14
    # two keys -> logistic weights
    K2 = np.array([[1.0, 0, 0, 0], [3.0, 0, 0, 0]])
    o2, _ = orc.attention(np.array([1.0, 0, 0, 0]), K2, V[:2], 1.0)
    w1 = 1.0 / (1.0 + math.exp(-2.0))
    np.testing.assert_allclose(o2, (1 - w1) * V[0] + w1 * V[1], rtol=1e-14)
    # one key far ahead -> that key's value
    K3 = np.array([[0.0, 0, 0, 0], [800.0, 0, 0, 0], [1.0, 0, 0, 0]])
    o3, _ = orc.attention(np.array([1.0, 0, 0, 0]), K3, V[:3], 1.0)
    np.testing.assert_allclose(o3, V[1], rtol=1e-15)
    # empty list
    o4, l4 = orc.attention(q, np.zeros((0, d)), np.zeros((0, d)), 1.0)
    assert np.all(o4 == 0) and l4 == -math.inf


def test_attention_hand_example(golden_dir):
    g = _golden(golden_dir, "hand_examples.txt")
    l = [0.0, math.log(2), math.log(4), math.log(2), 0.0, 0.0]
    K = np.array([[x, 0.0] for x in l])
    V = np.array([[float(j), 0.0] for j in range(6)])
    q = np.array([1.0, 0.0])
    kept = [int(x) for x in g["select_kept"]]
    o, _ = orc.attention(q, K[kept], V[kept], 1.0)
    assert abs(o[0] - float(Fraction(g["attend_kept"][0]))) < 1e-14
    o, lse = orc.attention(q, K, V, 1.0)
    assert abs(o[0] - float(Fraction(g["attend_full"][0]))) < 1e-14
    assert abs(lse - math.log(11)) < 1e-14
    assert o[1] == 0.0


def test_attention_invariants():
    rng = np.random.default_rng(3)
    L, d = 97, 32
    q, K, V = rng.standard_normal(d), rng.standard_normal((L, d)), rng.standard_normal((L, d))
    o, lse = orc.attention(q, K, V, 0.3)
    # permutation of the cache rows
    p = rng.permutation(L)
    o2, lse2 = orc.attention(q, K[p], V[p], 0.3)
    np.testing.assert_allclose(o2, o, rtol=1e-12, atol=1e-14)
    assert abs(lse - lse2) < 1e-12
    # any partition merged with the log-sum-exp rule equals the unsplit result
    for cuts in ([40], [1, 2, 96], [10, 30, 31, 80]):
        parts = np.split(np.arange(L), cuts)
        os_, ls_ = zip(*[orc.attention(q, K[i], V[i], 0.3) for i in parts])
        M = max(ls_)
        wts = np.array([math.exp(x - M) for x in ls_])
        merged = sum(w * o_ for w, o_ in zip(wts, os_)) / wts.sum()
        np.testing.assert_allclose(merged, o, rtol=1e-12, atol=1e-14)
        assert abs(M + math.log(wts.sum()) - lse) < 1e-12
    # shifting all logits leaves o unchanged and moves lse by the shift (q scaled keys)
    o3, lse3 = orc.attention(q, K, V + 1.0, 0.3)
    np.testing.assert_allclose(o3, o + 1.0, rtol=1e-12, atol=1e-12)


def test_decode_attention_gqa_mapping_and_append():
    rng = np.random.default_rng(4)
    B, Hq, Hkv, d = 2, 6, 2, 16
    lens = [[5, 9], [1, 0]]
    cache = orc.HybridCache(B, Hkv, d)
    for b in range(B):
        for h in range(Hkv):
            cache.k_rows.append(orc.f64_to_bf16(rng.standard_normal((lens[b][h], d))))
            cache.v_rows.append(orc.f64_to_bf16(rng.standard_normal((lens[b][h], d))))
    q = orc.f64_to_bf16(rng.standard_normal((B, Hq, d)))
    out, lse = orc.decode_attention(cache, q)
    G = Hq // Hkv
    for b, hq in itertools.product(range(B), range(Hq)):
        i = b * Hkv + hq // G
        K = orc.bf16_to_f64(cache.k_rows[i])
        V = orc.bf16_to_f64(cache.v_rows[i])
        if K.shape[0] == 0:
            assert np.all(out[b, hq] == 0) and lse[b, hq] == -math.inf
            continue
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(orc.bf16_to_f64(q[b, hq]))[None, None, None], torch.from_numpy(K)[None, None],
            torch.from_numpy(V)[None, None])[0, 0, 0].numpy()
        np.testing.assert_allclose(out[b, hq], ref, rtol=1e-12, atol=1e-14)
    # append: every list grows by exactly the new row, at its end
    kn = orc.f64_to_bf16(rng.standard_normal((B, Hkv, d)))
    vn = orc.f64_to_bf16(rng.standard_normal((B, Hkv, d)))
    before = [r.copy() for r in cache.k_rows]
    cache.append(kn, vn)
    for b in range(B):
        for h in range(Hkv):
            i = b * Hkv + h
            assert cache.k_rows[i].shape[0] == lens[b][h] + 1
            assert np.array_equal(cache.k_rows[i][:-1], before[i])
            assert np.array_equal(cache.k_rows[i][-1], kn[b, h])
            assert np.array_equal(cache.v_rows[i][-1], vn[b, h])
    assert list(cache.lengths()) == [6, 10, 2, 1]


def test_full_budget_reproduces_full_attention():
    # invariant: a budget equal to the full length keeps every token, in order,
    # so decode attention over the hybrid cache is full attention exactly
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=300, Hq=4, Hkv=2, budget=300)
    p = synth.prefill_layer(w, 0)
    qw, k, v = synth.bits(p["q_win"]), synth.bits(p["k"]), synth.bits(p["v"])
    mask = np.ones((1, 2), dtype=np.uint8)
    cache, idx = orc.select_compact(qw, k, v, p["seq_len"], mask, 300, 1.0, w.sink, w.local, w.L_obs,
                                    orc.POOL_NONE, 0)
    for i in idx:
        assert np.array_equal(i, np.arange(300))
    q, _, _ = synth.decode_inputs(w, 0, 0)
    out, _ = orc.decode_attention(cache, synth.bits(q))
    for hq in range(4):
        ref, _ = orc.attention(orc.bf16_to_f64(synth.bits(q)[0, hq]), orc.bf16_to_f64(k[0, hq // 2]),
                               orc.bf16_to_f64(v[0, hq // 2]), 1 / math.sqrt(128))
        assert np.array_equal(out[0, hq], ref)
