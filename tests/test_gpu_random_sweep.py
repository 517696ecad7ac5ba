"""GPU parity on seeded random shapes: many small caches with ragged lengths, random group sizes, CTA counts,
append schedules and selection parameters.  Each case is checked against the oracle like the targeted tests."""
import math

import numpy as np
import pytest
import torch

from oracle import catekv_oracle as orc
from workloads import synth
import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ck():
    import paper_2608_30295_b200 as pkg
    assert torch.cuda.is_available()
    return pkg.binding


@pytest.mark.parametrize("seed", range(12))
def test_random_decode_with_appends(ck, seed):
    rng = np.random.default_rng(1000 + seed)
    B, Hkv = int(rng.integers(1, 4)), int(rng.integers(1, 5))
    G = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8]))
    kinds = rng.integers(0, 4, size=B * Hkv)
    lens = [int({0: 0, 1: rng.integers(1, 70), 2: rng.integers(70, 700), 3: rng.integers(700, 6000)}[k]) for k in kinds]
    steps = int(rng.integers(1, 6))
    oc = H.random_cache(B, Hkv, lens, seed=2000 + seed)
    cache = H.device_cache_from_oracle(ck, oc, max_new=steps)
    plan = ck.DecodePlan(cache, int(rng.choice([1, 2, 7, 31, 296, 400])))
    ck.catekv_decode_plan(cache, plan)
    fused = bool(rng.integers(0, 2))
    o32 = torch.empty((B, Hkv * G, 128), dtype=torch.float32, device="cuda")
    o16 = torch.empty((B, Hkv * G, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hkv * G), dtype=torch.float32, device="cuda")
    scale = float(rng.choice([0.0, 0.05, 0.2]))
    for st in range(steps):
        kn = synth.randn_bf16((B, Hkv, 128), "cuda", 3000 + seed, "kn", st)
        vn = synth.randn_bf16((B, Hkv, 128), "cuda", 3000 + seed, "vn", st)
        q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 3000 + seed, "q", st)
        if fused:
            ck.catekv_append_decode_attn(cache, kn, vn, q, plan, o32, lse, sm_scale=scale)
        else:
            ck.catekv_append(cache, kn, vn)
            ck.catekv_decode_attn(cache, q, plan, o32, lse, sm_scale=scale)
        ck.catekv_decode_attn(cache, q, plan, o16, sm_scale=scale)
        oc.append(synth.bits(kn), synth.bits(vn))
        ref, ref_lse = orc.decode_attention(oc, synth.bits(q), scale=scale if scale else None)
        H.check_attention(o32, o16, lse, ref, ref_lse, f"seed {seed} step {st} lens {lens} G {G} fused {fused}")
    assert cache.seg_len_dev.cpu().tolist() == [l + steps for l in lens]


@pytest.mark.parametrize("seed", range(8))
def test_random_select(ck, seed):
    rng = np.random.default_rng(4000 + seed)
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 7]))
    L_obs = int(rng.choice([8, 16, 32, 33, 64]))
    local = L_obs + int(rng.integers(0, 40))
    sink = int(rng.integers(0, 9))
    B = int(rng.integers(1, 3))
    n = int(rng.integers(local + sink + 40, 1800))
    w = synth.scaled(synth.WORKLOADS["cfg0"], B=B, Hq=Hkv * G, Hkv=Hkv, n=n, L_obs=L_obs, sink=sink, local=local,
                     seed=5000 + seed)
    p = synth.prefill_layer(w, 0)
    seq_len = [n] + [int(rng.integers(local + sink + 20, n + 1)) for _ in range(B - 1)]
    mask = rng.integers(0, 3, size=(B, Hkv)).astype(np.uint8)
    budget = int(rng.integers(sink + local, n))
    eta = float(rng.choice([1.0, 0.9, 0.5]))
    mode, param = [(orc.POOL_NONE, 0), (orc.POOL_SLIDING, 7), (orc.POOL_SLIDING, 3), (orc.POOL_CHUNK, 8),
                   (orc.POOL_CHUNK, 3)][int(rng.integers(0, 5))]
    eta32 = float(np.float32(eta))
    ub = []
    for b in range(B):
        for h in range(Hkv):
            T = orc.token_budget(seq_len[b], int(mask[b, h]), budget, eta32, sink, local)
            ub.append(seq_len[b] if (T >= seq_len[b] or sink + local >= seq_len[b]) else max(T, sink + local))
    cache = ck.Cache(B, Hkv, ub, 0, "cuda")
    idx = torch.full((B * Hkv, n), -1, dtype=torch.int32, device="cuda")
    ck.catekv_select_compact(p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda(), seq_len, mask, cache, budget, eta, sink,
                             local, mode, param, idx_out=idx)
    torch.cuda.synchronize()
    idx = idx.cpu().numpy()
    qw, k, v = synth.bits(p["q_win"]), synth.bits(p["k"]), synth.bits(p["v"])
    kp, vp = synth.bits(cache.k_pool), synth.bits(cache.v_pool)
    assert np.array_equal(cache.seg_len_dev.cpu().numpy(), cache.seg_len)
    for b in range(B):
        nb = seq_len[b]
        for h in range(Hkv):
            i = b * Hkv + h
            T = orc.token_budget(nb, int(mask[b, h]), budget, eta32, sink, local)
            L = int(cache.seg_len[i])
            got = idx[i, :L]
            where = f"seed {seed} b{b} h{h} n{nb} T{T} mode{mode}/{param} G{G} L_obs{L_obs}"
            if T >= nb or sink + local >= nb:
                assert np.array_equal(got, np.arange(nb)), where
            else:
                C = orc.window_scores(qw[b, h * G:(h + 1) * G], k[b, h, :nb], L_obs)
                H.check_indices_band(got, C, nb, sink, local, T, mode, param, where)
            o = int(cache.seg_off[i])
            assert np.array_equal(kp[o:o + L], k[b, h][got]) and np.array_equal(vp[o:o + L], v[b, h][got]), where
