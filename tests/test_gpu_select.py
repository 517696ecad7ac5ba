"""GPU parity: catekv_select_compact against the CPU oracle (indices, layout, lengths)."""
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


def _select(ck, w, p, mask, budget, eta, mode, param, max_new=0, seq_len=None):
    seq_len = p["seq_len"] if seq_len is None else np.asarray(seq_len, dtype=np.int32)
    eta32 = float(np.float32(eta))
    len_ub = []
    for b in range(w.B):
        n = int(seq_len[b])
        for h in range(w.Hkv):
            T = orc.token_budget(n, bool(mask[b, h]), budget, eta32)
            len_ub.append(n if (T >= n or w.sink + w.local >= n) else min(n, max(T, w.sink + w.local)))
    cache = ck.Cache(w.B, w.Hkv, len_ub, max_new, "cuda")
    idx = torch.full((w.B * w.Hkv, w.n), -1, dtype=torch.int32, device="cuda")
    ck.catekv_select_compact(p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda(), seq_len, mask, cache, budget, eta,
                             w.sink, w.local, mode, param, idx_out=idx)
    if cache.struct.reserved:  # chunk mode with a short last chunk: the host lengths are upper bounds until synced
        bound = cache.seg_len.copy()
        ck.catekv_cache_sync_lengths(cache)
        assert np.all(cache.seg_len <= bound) and np.all(bound - cache.seg_len < max(param, 1))
        assert cache.struct.reserved == 0
    torch.cuda.synchronize()
    return cache, idx.cpu().numpy()


def _check_against_oracle(ck, w, p, mask, budget, eta, mode, param, seq_len=None, cells=None):
    seq_len = p["seq_len"] if seq_len is None else np.asarray(seq_len, dtype=np.int32)
    cache, idx = _select(ck, w, p, mask, budget, eta, mode, param, seq_len=seq_len)
    qw, k, v = synth.bits(p["q_win"]), synth.bits(p["k"]), synth.bits(p["v"])
    eta32 = float(np.float32(eta))
    exact = 0
    dev_len = cache.seg_len_dev.cpu().numpy()
    kp, vp = synth.bits(cache.k_pool), synth.bits(cache.v_pool)
    todo = cells if cells is not None else [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    for (b, h) in todo:
        n = int(seq_len[b])
        i = b * w.Hkv + h
        T = orc.token_budget(n, bool(mask[b, h]), budget, eta32)
        L = int(cache.seg_len[i])
        assert L == dev_len[i]
        got = idx[i, :L]
        if T >= n or w.sink + w.local >= n:
            assert np.array_equal(got, np.arange(n))
        else:
            C = orc.window_scores(qw[b, h * w.G:(h + 1) * w.G], k[b, h, :n], w.L_obs)
            exact += H.check_indices_band(got, C, n, w.sink, w.local, T, mode, param, f"b{b} h{h}")
        # the segment holds exactly the rows of its own index list, in that order
        o = int(cache.seg_off[i])
        assert np.array_equal(kp[o:o + L], k[b, h][got]), (b, h)
        assert np.array_equal(vp[o:o + L], v[b, h][got]), (b, h)
    return cache, idx, exact


def test_select_planted_only_is_bit_exact(ck):
    # k_rest = 16 = the planted heavy keys: the score gap at the threshold is wide, so indices are exact
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=2048)
    p = synth.prefill_layer(w, 0)
    budget = w.sink + w.local + synth.N_HEAVY
    cache, idx, exact = _check_against_oracle(ck, w, p, p["head_mask"], budget, 1.0, orc.POOL_NONE, 0)
    assert exact == int(p["head_mask"].sum())
    for h in range(w.Hkv):
        if p["head_mask"][0, h]:
            assert set(p["heavy"][0, h]) <= set(idx[h, :budget].tolist())


@pytest.mark.parametrize("mode,param", [(orc.POOL_NONE, 0), (orc.POOL_SLIDING, 7), (orc.POOL_CHUNK, 8),
                                        (orc.POOL_SLIDING, 1), (orc.POOL_CHUNK, 1), (orc.POOL_CHUNK, 5)])
def test_select_cfg0_all_modes(ck, mode, param):
    w = synth.WORKLOADS["cfg0"]
    p = synth.prefill_layer(w, 0)
    _check_against_oracle(ck, w, p, p["head_mask"], w.budget, 1.0, mode, param)


@pytest.mark.parametrize("Hq,Hkv,L_obs", [(8, 8, 16), (28, 4, 64), (16, 2, 48), (6, 2, 7), (16, 2, 64), (10, 2, 50)])
def test_select_shapes_and_adaptive_eta(ck, Hq, Hkv, L_obs):
    w = synth.scaled(synth.WORKLOADS["cfg0"], Hq=Hq, Hkv=Hkv, L_obs=L_obs, n=1500, B=2)
    p = synth.prefill_layer(w, 1)
    mask = p["head_mask"]
    # ragged sequence lengths inside one batch; adaptive heads keep 90 %
    _check_against_oracle(ck, w, p, mask, 200, 0.9, orc.POOL_SLIDING, 7, seq_len=[1500, 1111])
    _check_against_oracle(ck, w, p, mask, 200, 0.9, orc.POOL_CHUNK, 8, seq_len=[1500, 1111])


def test_select_degenerate_budgets(ck):
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=300, Hq=8, Hkv=2)
    p = synth.prefill_layer(w, 2)
    mask = np.ones((1, 2), dtype=np.uint8)
    # budget >= n: everything; budget == sink + local: no top-k slot; budget below that: still sink + local
    for budget in (300, 5000, w.sink + w.local, 10, 0, w.sink + w.local + 1, 299):
        cache, idx, _ = _check_against_oracle(ck, w, p, mask, budget, 1.0, orc.POOL_NONE, 0)
        want = 300 if budget >= 300 else max(budget, w.sink + w.local)
        assert list(cache.seg_len) == [want, want]
    # a sequence shorter than sink + local keeps everything
    _check_against_oracle(ck, w, p, mask, 40, 1.0, orc.POOL_SLIDING, 3, seq_len=[60])
    # chunk budget smaller than one chunk: nothing selected
    _check_against_oracle(ck, w, p, mask, w.sink + w.local + 7, 1.0, orc.POOL_CHUNK, 8)


def test_select_ties_lowest_index(ck):
    # identical keys give exactly equal scores: the selection must be the first k_rest candidates
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=400, Hq=4, Hkv=1)
    p = synth.prefill_layer(w, 3)
    p["k"][:, :, : w.n - w.L_obs] = p["k"][:, :, :1]
    mask = np.ones((1, 1), dtype=np.uint8)
    for mode, param in ((orc.POOL_NONE, 0), (orc.POOL_SLIDING, 7), (orc.POOL_CHUNK, 8)):
        cache, idx, _ = _check_against_oracle(ck, w, p, mask, 128, 1.0, mode, param)
        L = int(cache.seg_len[0])
        k_rest = 128 - w.sink - w.local
        if mode == orc.POOL_CHUNK:
            k_rest = k_rest // 8 * 8
        assert list(idx[0, :w.sink + k_rest]) == list(range(w.sink + k_rest))


def test_select_then_decode_end_to_end_cfg0(ck):
    # configs[0]: 4 of 8 KV heads consistent at 256 = 4 + 64 + 188, 16 decode steps
    w = synth.WORKLOADS["cfg0"]
    p = synth.prefill_layer(w, 0)
    mask = p["head_mask"]
    assert int(mask.sum()) == 4
    cache, idx = _select(ck, w, p, mask, w.budget, w.eta, w.pool_mode, w.pool_param, max_new=w.decode_steps)
    # the oracle continues from the device's own kept lists (bit-exact layout), so that decode parity
    # is not blurred by near-tie differences in the selection
    oc = orc.HybridCache(w.B, w.Hkv, w.d)
    k, v = synth.bits(p["k"]), synth.bits(p["v"])
    for h in range(w.Hkv):
        L = int(cache.seg_len[h])
        assert L == (w.budget if mask[0, h] else w.n)
        oc.k_rows.append(k[0, h][idx[h, :L]])
        oc.v_rows.append(v[0, h][idx[h, :L]])
    plan = ck.DecodePlan(cache, ck.catekv_decode_num_ctas())
    ck.catekv_decode_plan(cache, plan)
    o32 = torch.empty((w.B, w.Hq, w.d), dtype=torch.float32, device="cuda")
    o16 = torch.empty((w.B, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.B, w.Hq), dtype=torch.float32, device="cuda")
    for step in range(w.decode_steps):
        q, kn, vn = synth.decode_inputs(w, 0, step, "cpu", mask)
        ck.catekv_append(cache, kn.cuda(), vn.cuda())
        oc.append(synth.bits(kn), synth.bits(vn))
        ck.catekv_decode_attn(cache, q.cuda(), plan, o32, lse)
        ck.catekv_decode_attn(cache, q.cuda(), plan, o16)
        ref, ref_lse = orc.decode_attention(oc, synth.bits(q))
        H.check_attention(o32, o16, lse, ref, ref_lse, f"step {step}")
    # and fully independently: oracle selection -> oracle decode, compared on the heads whose lists agree
    oc2, oidx = orc.select_compact(synth.bits(p["q_win"]), k, v, p["seq_len"], mask, w.budget, w.eta, w.sink,
                                   w.local, w.L_obs, w.pool_mode, w.pool_param)
    same = [h for h in range(w.Hkv) if np.array_equal(oidx[h], idx[h, :len(oidx[h])])]
    assert len(same) >= 4  # at least every adaptive head


def test_select_full_budget_equals_full_attention(ck):
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=700, Hq=8, Hkv=2)
    p = synth.prefill_layer(w, 4)
    mask = np.ones((1, 2), dtype=np.uint8)
    cache, idx = _select(ck, w, p, mask, 700, 1.0, orc.POOL_NONE, 0)
    plan = ck.DecodePlan(cache, 6)
    ck.catekv_decode_plan(cache, plan)
    q, _, _ = synth.decode_inputs(w, 4, 0, "cpu", mask)
    out = torch.empty((1, 8, 128), dtype=torch.float32, device="cuda")
    ck.catekv_decode_attn(cache, q.cuda(), plan, out)
    k, v, qb = synth.bits(p["k"]), synth.bits(p["v"]), synth.bits(q)
    ref = np.stack([orc.attention(orc.bf16_to_f64(qb[0, hq]), orc.bf16_to_f64(k[0, hq // 4]),
                                  orc.bf16_to_f64(v[0, hq // 4]), 1 / math.sqrt(128))[0] for hq in range(8)])
    H.check_attention(out[0], None, None, ref, None)


def test_streaming_heads_and_attention_recall(ck):
    # three head types in one launch; recall of each kept set against the oracle's definition
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=3000, Hq=24, Hkv=6)
    p = synth.prefill_layer(w, 6)
    mask = np.array([[2, 1, 0, 1, 2, 0]], dtype=np.uint8)
    lens = [w.sink + w.local, 256, w.n, 256, w.sink + w.local, w.n]
    cache = ck.Cache(1, 6, lens, 4, "cuda")
    full = ck.Cache(1, 6, [w.n] * 6, 4, "cuda")
    idx = torch.full((6, w.n), -1, dtype=torch.int32, device="cuda")
    args = (p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda(), p["seq_len"])
    ck.catekv_select_compact(*args, mask, cache, 256, 1.0, w.sink, w.local, orc.POOL_SLIDING, 7, idx_out=idx)
    ck.catekv_select_compact(*args, np.zeros((1, 6), dtype=np.uint8), full, 256, 1.0, w.sink, w.local, orc.POOL_NONE, 0)
    torch.cuda.synchronize()
    assert list(cache.seg_len) == lens and list(full.seg_len) == [w.n] * 6
    idx = idx.cpu().numpy()
    for h in (0, 4):
        assert list(idx[h, :lens[h]]) == list(range(w.sink)) + list(range(w.n - w.local, w.n))
    q, _, _ = synth.decode_inputs(w, 6, 0, "cpu", (mask == 1).astype(np.uint8))
    plan, plan_f = ck.DecodePlan(cache, 8), ck.DecodePlan(full, 8)
    ck.catekv_decode_plan(cache, plan)
    ck.catekv_decode_plan(full, plan_f)
    out = torch.empty((1, 24, 128), dtype=torch.float32, device="cuda")
    lse_k = torch.empty((1, 24), dtype=torch.float32, device="cuda")
    lse_f = torch.empty_like(lse_k)
    ck.catekv_decode_attn(cache, q.cuda(), plan, out, lse_k)
    ck.catekv_decode_attn(full, q.cuda(), plan_f, out, lse_f)
    rec = ck.catekv_attention_recall(lse_k, lse_f).cpu().numpy()[0]
    kb, qb = synth.bits(p["k"]), synth.bits(q)
    for hq in range(24):
        h = hq // 4
        want = orc.attention_recall(orc.bf16_to_f64(qb[0, hq]), orc.bf16_to_f64(kb[0, h]), idx[h, :lens[h]],
                                    1 / math.sqrt(128))
        assert rec[hq] == pytest.approx(want, rel=2e-3, abs=1e-6), (hq, rec[hq], want)
    assert np.allclose(rec[8:12], 1.0, atol=1e-4) and np.allclose(rec[20:24], 1.0, atol=1e-4)  # adaptive: everything kept
    # consistent heads lean on their planted keys: they recall more mass than the streaming heads of this input
    assert rec[4:8].mean() > rec[0:4].mean()


def test_token_major_kv_layout_gives_identical_results(ck):
    """K and V as [B, n, Hkv, d] views (token-major storage, the head stride smaller than the token stride): the
    strides go into the tensor map and the gather; selection, window attention and the CV score must not change a bit."""
    w = synth.scaled(synth.WORKLOADS["cfg0"], B=2, n=1500, budget=200, seed=77)
    p = synth.prefill_layer(w, 0)
    mask = p["head_mask"]
    qw, k, v = p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda()
    kt = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)   # same values, strides (n*Hkv*d, d, Hkv*d, 1)
    vt = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert kt.stride() != k.stride() and torch.equal(kt, k)
    seq_len = [w.n, 1203]
    lens = []
    for b in range(w.B):
        lens += [w.budget if mask[b, h] else seq_len[b] for h in range(w.Hkv)]
    res = []
    for kk, vv in ((k, v), (kt, vt)):
        cache = ck.Cache(w.B, w.Hkv, lens, 0, "cuda")
        idx = torch.full((w.B * w.Hkv, w.n), -1, dtype=torch.int32, device="cuda")
        ck.catekv_select_compact(qw, kk, vv, seq_len, mask, cache, w.budget, 1.0, w.sink, w.local, orc.POOL_SLIDING, 7,
                                 idx_out=idx)
        wa = ck.catekv_window_attn(qw, kk, vv, seq_len)
        cv = ck.catekv_head_cv(qw, kk, seq_len, 16, 40, 0.99, 1.0, True)
        torch.cuda.synchronize()
        res.append((cache.seg_len.copy(), idx.clone(), cache.k_pool.clone(), cache.v_pool.clone(), wa, cv))
    a, b = res
    assert np.array_equal(a[0], b[0]) and torch.equal(a[1], b[1])
    for s in range(w.B * w.Hkv):
        o, L = int(ck.catekv_cache_layout(w.B, w.Hkv, lens, 0)[0][s]), int(a[0][s])
        assert torch.equal(a[2][o:o + L], b[2][o:o + L]) and torch.equal(a[3][o:o + L], b[3][o:o + L])
    for x, y in zip(a[4], b[4]):
        assert torch.equal(x, y)
    assert torch.equal(a[5], b[5])
