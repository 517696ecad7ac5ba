"""GPU parity at the full sizes of the five configurations, in the launch configuration bench.py times
(plan over SMs x resident CTAs, caches built by catekv_select_compact).  The oracle is run on sampled
(sequence, KV head) cells: their prefill rows and kept lists are copied back and checked one by one."""
import math

import numpy as np
import pytest
import torch

from oracle import catekv_oracle as orc
from workloads import synth
import helpers as H
import bench

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ck():
    import paper_2608_30295_b200 as pkg
    assert torch.cuda.is_available()
    return pkg.binding


def _build_layer(ck, w, layer, max_new):
    p = synth.prefill_layer(w, layer, "cuda")
    mask = p["head_mask"]
    cache = ck.Cache(w.B, w.Hkv, bench.expected_lengths(w, mask), max_new, "cuda")
    idx = torch.full((w.B * w.Hkv, w.n), -1, dtype=torch.int32, device="cuda")
    ck.catekv_select_compact(p["q_win"], p["k"], p["v"], p["seq_len"], mask, cache, w.budget, w.eta, w.sink, w.local,
                             w.pool_mode, w.pool_param, idx_out=idx)
    if cache.struct.reserved:  # chunk mode, short last chunk: exact lengths for the fused-append path and the checks
        ck.catekv_cache_sync_lengths(cache)
    torch.cuda.synchronize()
    return p, mask, cache, idx


def _check_selection_cells(w, p, mask, cache, idx, cells):
    """Selected indices (band-aware) and segment bytes of the sampled cells; returns oracle caches of the cells
    built from the device's own kept lists."""
    eta32 = float(np.float32(w.eta))
    oc = orc.HybridCache(w.B, w.Hkv, w.d)
    oc.k_rows = [np.zeros((0, w.d), dtype=np.uint16)] * (w.B * w.Hkv)
    oc.v_rows = [np.zeros((0, w.d), dtype=np.uint16)] * (w.B * w.Hkv)
    dev_len = cache.seg_len_dev.cpu().numpy()
    assert np.array_equal(dev_len, cache.seg_len)
    for (b, h) in cells:
        i = b * w.Hkv + h
        L = int(cache.seg_len[i])
        got = idx[i, :L].cpu().numpy()
        k = synth.bits(p["k"][b, h])
        v = synth.bits(p["v"][b, h])
        T = orc.token_budget(w.n, bool(mask[b, h]), w.budget, eta32)
        if T >= w.n:
            assert np.array_equal(got, np.arange(w.n))
        else:
            qw = synth.bits(p["q_win"][b, h * w.G:(h + 1) * w.G])
            C = orc.window_scores(qw, k, w.L_obs)
            H.check_indices_band(got, C, w.n, w.sink, w.local, T, w.pool_mode, w.pool_param, f"{w.name} b{b} h{h}")
            assert L == min(w.n, T) or w.pool_mode == orc.POOL_CHUNK
            # every planted heavy key is far above the threshold
            assert set(p["heavy"][b, h]) <= set(got.tolist())
        o = int(cache.seg_off[i])
        assert np.array_equal(synth.bits(cache.k_pool[o:o + L]), k[got])
        assert np.array_equal(synth.bits(cache.v_pool[o:o + L]), v[got])
        oc.k_rows[i] = k[got]
        oc.v_rows[i] = v[got]
    return oc


def _decode_steps(ck, w, layer, mask, cache, oc, cells, n_steps, check_steps):
    plan = ck.DecodePlan(cache, ck.catekv_decode_num_ctas())
    ck.catekv_decode_plan(cache, plan)
    o32 = torch.empty((w.B, w.Hq, w.d), dtype=torch.float32, device="cuda")
    o16 = torch.empty((w.B, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.B, w.Hq), dtype=torch.float32, device="cuda")
    for step in range(n_steps):
        q, kn, vn = synth.decode_inputs(w, layer, step, "cuda", mask)
        ck.catekv_append(cache, kn, vn)
        knb, vnb = synth.bits(kn), synth.bits(vn)
        for (b, h) in cells:
            i = b * w.Hkv + h
            oc.k_rows[i] = np.concatenate([oc.k_rows[i], knb[b, h][None]])
            oc.v_rows[i] = np.concatenate([oc.v_rows[i], vnb[b, h][None]])
        if step in check_steps:
            ck.catekv_decode_attn(cache, q, plan, o32, lse)
            ck.catekv_decode_attn(cache, q, plan, o16)
            ref, ref_lse = orc.decode_attention(oc, synth.bits(q), cells=cells)
            H.check_attention(o32, o16, lse, ref, ref_lse, f"{w.name} layer {layer} step {step}")


def _pick_cells(mask, want):
    """Up to `want` cells, alternating consistent and adaptive heads across sequences."""
    cons = [(b, h) for b in range(mask.shape[0]) for h in range(mask.shape[1]) if mask[b, h]]
    adap = [(b, h) for b in range(mask.shape[0]) for h in range(mask.shape[1]) if not mask[b, h]]
    rng = np.random.default_rng(int(mask.sum()) + 7)
    rng.shuffle(cons), rng.shuffle(adap)
    out = []
    while len(out) < want and (cons or adap):
        if cons:
            out.append(cons.pop())
        if adap and len(out) < want:
            out.append(adap.pop())
    return out


def test_cfg1_32k_four_layers_steps_0_1_127(ck):
    w = synth.WORKLOADS["cfg1"]
    for layer in (0, 9, 17, 31):
        p, mask, cache, idx = _build_layer(ck, w, layer, w.decode_steps)
        cells = _pick_cells(mask, 4)
        oc = _check_selection_cells(w, p, mask, cache, idx, cells)
        del p, idx
        _decode_steps(ck, w, layer, mask, cache, oc, cells, 128, {0, 1, 127})
        assert np.all(cache.seg_len_dev.cpu().numpy() == cache.seg_len)


def test_cfg2_128k_adaptive_keeps_90_percent(ck):
    w = synth.WORKLOADS["cfg2"]
    p, mask, cache, idx = _build_layer(ck, w, 3, 8)
    lens = cache.seg_len.reshape(w.B, w.Hkv)
    assert set(np.unique(lens[mask == 1])) <= {2048} and set(np.unique(lens[mask == 0])) == {117964}
    cells = _pick_cells(mask, 3)
    oc = _check_selection_cells(w, p, mask, cache, idx, cells)
    del p, idx
    _decode_steps(ck, w, 3, mask, cache, oc, cells, 3, {0, 1, 2})


def test_cfg3_batch16_ragged_masks(ck):
    w = synth.WORKLOADS["cfg3"]
    p, mask, cache, idx = _build_layer(ck, w, 5, 8)
    per_seq = mask.sum(axis=1)
    assert per_seq.min() >= 3 and per_seq.max() <= 6 and len(set(per_seq.tolist())) > 1  # 40-70 % of 8 heads
    cells = _pick_cells(mask, 4)
    assert len({b for b, _ in cells}) >= 3
    oc = _check_selection_cells(w, p, mask, cache, idx, cells)
    del p, idx
    _decode_steps(ck, w, 5, mask, cache, oc, cells, 2, {0, 1})


def test_cfg4_qwen_gqa7_chunks(ck):
    w = synth.WORKLOADS["cfg4"]
    p, mask, cache, idx = _build_layer(ck, w, 2, 8)
    cells = _pick_cells(mask, 2)
    oc = _check_selection_cells(w, p, mask, cache, idx, cells)
    del p, idx
    _decode_steps(ck, w, 2, mask, cache, oc, cells, 2, {0, 1})


def test_cfg4_head_mask_from_calibration_prompts(ck):
    # 8 calibration prompts of 16K tokens; the library's scores and vote must reproduce the oracle's mask
    w = synth.WORKLOADS["cfg4"]
    layers, prompts, n = 4, 8, 16384
    L_init, L_rec = 2048 // 32, 2048 // 128
    rng = np.random.default_rng(44)
    types = np.stack([rng.permutation(np.array([1, 1, 0, 0], dtype=np.uint8)) for _ in range(layers)])
    got = np.zeros((prompts, layers * w.Hkv), dtype=np.float32)
    want = np.zeros((prompts, layers * w.Hkv))
    for l in range(layers):
        qs, ks = zip(*[synth.calibration_prompt(w, l, pr, n, types[l], "cuda") for pr in range(prompts)])
        q, k = torch.cat(qs), torch.cat(ks)
        cv = ck.catekv_head_cv(q, k, [n] * prompts, L_init, L_rec, 0.99, 1.0, True).cpu().numpy()
        got[:, l * w.Hkv:(l + 1) * w.Hkv] = cv
        ref = orc.head_cv(synth.bits(q), synth.bits(k), [n] * prompts, w.L_obs, L_init, L_rec,
                          float(np.float32(0.99)), 1.0, True)
        want[:, l * w.Hkv:(l + 1) * w.Hkv] = ref
    np.testing.assert_allclose(got, want, rtol=1e-3)
    m = ck.catekv_classify_heads(got, 0.5)
    assert np.array_equal(m, orc.static_head_mask(want, 0.5))
    assert np.array_equal(m, types.reshape(-1))


def test_cfg2_retrieval_on_adaptive_heads(ck):
    # configs[2] shape: adaptive heads (117 964 rows) answer a decode query from 2048 retrieved rows, chunk size 8
    w = synth.WORKLOADS["cfg2"]
    p, mask, cache, idx = _build_layer(ck, w, 3, 8)
    cs, budget = 8, 2048
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    q, kn, vn = synth.decode_inputs(w, 3, 0, "cuda", mask)
    ck.catekv_append(cache, kn, vn)
    ck.catekv_retrieval_append(cache, cs, kn, meta)
    rmask = (mask.reshape(-1) == 0).astype(np.uint8)
    lens = [int(L) for L in cache.seg_len]
    slens = [len(orc.retrieve_indices(np.zeros((L + cs - 1) // cs), L, w.sink, w.local, budget, cs)) if rmask[i] else L
             for i, L in enumerate(lens)]
    step = ck.Cache(w.B, w.Hkv, slens, 0, "cuda")
    ridx = torch.full((w.B * w.Hkv, max(lens)), -1, dtype=torch.int32, device="cuda")
    ck.catekv_retrieve_compact(cache, meta, cs, q, rmask, budget, w.sink, w.local, step, idx_out=ridx)
    torch.cuda.synchronize()
    assert list(step.seg_len) == slens
    cells = [int(i) for i in np.nonzero(rmask)[0][:2]] + [int(np.nonzero(rmask == 0)[0][0])]
    qb = orc.bf16_to_f64(synth.bits(q))
    soc = orc.HybridCache(w.B, w.Hkv, w.d)
    soc.k_rows = [np.zeros((0, w.d), dtype=np.uint16)] * (w.B * w.Hkv)
    soc.v_rows = [np.zeros((0, w.d), dtype=np.uint16)] * (w.B * w.Hkv)
    for s in cells:
        o, L = int(cache.seg_off[s]), lens[s]
        krows, vrows = synth.bits(cache.k_pool[o:o + L]), synth.bits(cache.v_pool[o:o + L])
        got = ridx[s, :slens[s]].cpu().numpy().astype(np.int64)
        if rmask[s]:
            kmax, kmin = orc.retrieval_metadata(krows, cs)
            scores = orc.retrieval_scores(qb[0, s * w.G:(s + 1) * w.G], kmax, kmin)
            H.check_retrieval_band(got, scores, L, w.sink, w.local, budget, cs, f"cfg2 seg {s}")
        else:
            assert np.array_equal(got, np.arange(L))
        so = int(step.seg_off[s])
        assert np.array_equal(synth.bits(step.k_pool[so:so + slens[s]]), krows[got])
        soc.k_rows[s], soc.v_rows[s] = krows[got], vrows[got]
    plan = ck.DecodePlan(step, ck.catekv_decode_num_ctas())
    ck.catekv_decode_plan(step, plan)
    out = torch.empty((w.B, w.Hq, w.d), dtype=torch.float32, device="cuda")
    ck.catekv_decode_attn(step, q, plan, out)
    ref, _ = orc.decode_attention(soc, synth.bits(q), cells=[(0, s) for s in cells])
    H.check_attention(out, None, None, ref, None, "cfg2 retrieval")


def test_cfg3_retrieval_in_place_as_the_bench_runs_it(ck):
    # configs[3] shape, the retrieval step bench.py times: 1024 rows per adaptive head, chunk size 8, one-launch
    # append, index lists, attention in place under a plan over all resident CTAs
    w = synth.WORKLOADS["cfg3"]
    layer, cs, budget = 7, 8, 1024
    p, mask, cache, idx = _build_layer(ck, w, layer, 8)
    del p, idx
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    rmask = (mask.reshape(-1) == 0).astype(np.uint8)
    n_segs = w.B * w.Hkv
    ridx = torch.full((n_segs, budget + 2 * cs + w.local), -1, dtype=torch.int32, device="cuda")
    sel = torch.full((n_segs,), -99, dtype=torch.int32, device="cuda")
    view = ck.CacheView(cache, ck.catekv_retrieve_lengths(cache, cs, rmask, budget, w.sink, w.local))
    plan = ck.DecodePlan(view, ck.catekv_decode_num_ctas())
    ck.catekv_decode_plan(view, plan)
    out = torch.empty((w.B, w.Hq, w.d), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.B, w.Hq), dtype=torch.float32, device="cuda")
    for step in range(2):
        q, kn, vn = synth.decode_inputs(w, layer, step, "cuda", mask)
        ck.catekv_append_retrieval(cache, kn, vn, cs, meta)
        ck.catekv_retrieve_select(cache, meta, cs, q, rmask, budget, w.sink, w.local, ridx, sel)
        ck.catekv_decode_attn_indexed(cache, ridx, sel, q, plan, out, lse)
    torch.cuda.synchronize()
    lens = [int(L) for L in cache.seg_len]
    got_sel = sel.cpu().tolist()
    want_len = ck.catekv_retrieve_lengths(cache, cs, rmask, budget, w.sink, w.local)
    ret = np.nonzero(rmask)[0]
    cells = [int(ret[0]), int(ret[len(ret) // 2]), int(ret[-1]), int(np.nonzero(rmask == 0)[0][3])]
    qb = orc.bf16_to_f64(synth.bits(q))
    soc = orc.HybridCache(w.B, w.Hkv, w.d)
    soc.k_rows = [np.zeros((0, w.d), dtype=np.uint16)] * n_segs
    soc.v_rows = [np.zeros((0, w.d), dtype=np.uint16)] * n_segs
    for s in cells:
        o, L = int(cache.seg_off[s]), lens[s]
        krows, vrows = synth.bits(cache.k_pool[o:o + L]), synth.bits(cache.v_pool[o:o + L])
        b, h = divmod(s, w.Hkv)
        if rmask[s]:
            assert got_sel[s] == want_len[s] and want_len[s] <= budget
            got = ridx[s, :got_sel[s]].cpu().numpy().astype(np.int64)
            kmax, kmin = orc.retrieval_metadata(krows, cs)
            # the metadata the device keeps, appended rows included
            c0 = o // cs
            m = synth.bits(meta.view(torch.bfloat16).view(-1, 2, 128)[c0:c0 + kmax.shape[0]])
            assert np.array_equal(orc.bf16_to_f64(m[:, 0]), kmax) and np.array_equal(orc.bf16_to_f64(m[:, 1]), kmin)
            scores = orc.retrieval_scores(qb[b, h * w.G:(h + 1) * w.G], kmax, kmin)
            H.check_retrieval_band(got, scores, L, w.sink, w.local, budget, cs, f"cfg3 seg {s}")
        else:
            assert got_sel[s] == -1
            got = np.arange(L)
        soc.k_rows[s], soc.v_rows[s] = krows[got], vrows[got]
    ref, ref_lse = orc.decode_attention(soc, synth.bits(q), cells=[divmod(s, w.Hkv) for s in cells])
    H.check_attention(out, None, lse, ref, ref_lse, "cfg3 retrieval in place")


def test_cfg2_window_attention_and_selection_from_its_normaliser(ck):
    # configs[2] shape (128K keys, 4 x 32 window rows per KV head): the prefill rows of the window, their normalisers,
    # and catekv_select_compact fed with them instead of running its own first pass over K
    w = synth.WORKLOADS["cfg2"]
    p = synth.prefill_layer(w, 1, "cuda")
    mask = p["head_mask"]
    out, lse, lse_sc = ck.catekv_window_attn(p["q_win"], p["k"], p["v"], p["seq_len"])
    out16, _, _ = ck.catekv_window_attn(p["q_win"], p["k"], p["v"], p["seq_len"], out_dtype=torch.bfloat16)
    cells = _pick_cells(mask, 2)
    qb = synth.bits(p["q_win"])
    for (b, h) in cells:
        kb, vb = synth.bits(p["k"][b, h]), synth.bits(p["v"][b, h])
        sl = slice(h * w.G, (h + 1) * w.G)
        ref, ref_lse = orc.window_attention(qb[b, sl], kb, vb, w.L_obs)
        H.check_attention(out[b, sl].reshape(-1, w.d), out16[b, sl].reshape(-1, w.d), lse[b, sl].reshape(-1),
                          ref.reshape(-1, w.d), ref_lse.reshape(-1), f"cfg2 window b{b} h{h}")
        ref_sc = orc.scored_range_lse(qb[b, sl], kb, w.L_obs)
        assert np.all(np.abs(lse_sc[b, sl].cpu().double().numpy() - ref_sc) <= 1e-3)
    cache = ck.Cache(w.B, w.Hkv, bench.expected_lengths(w, mask), 8, "cuda")
    idx = torch.full((w.B * w.Hkv, w.n), -1, dtype=torch.int32, device="cuda")
    ck.catekv_select_compact(p["q_win"], p["k"], p["v"], p["seq_len"], mask, cache, w.budget, w.eta, w.sink, w.local,
                             w.pool_mode, w.pool_param, idx_out=idx, row_lse_scored=lse_sc)
    torch.cuda.synchronize()
    _check_selection_cells(w, p, mask, cache, idx, cells)


def test_cfg4_window_attention_sampled_heads(ck):
    # configs[4] shape: 256K keys, 7 x 64 = 448 window rows per KV head (four 128-row tiles, the last one half
    # full, nine key ranges per tile).  The oracle checks the rows of three sampled query heads one by one.
    w = synth.WORKLOADS["cfg4"]
    p = synth.prefill_layer(w, 0, "cuda")
    out, lse, lse_sc = ck.catekv_window_attn(p["q_win"], p["k"], p["v"], p["seq_len"])
    out16, _, _ = ck.catekv_window_attn(p["q_win"], p["k"], p["v"], p["seq_len"], out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    qb = synth.bits(p["q_win"])
    for (b, hq) in [(0, 0), (1, 13), (3, 27)]:  # first, a middle and the last head (the last rows of a last tile)
        h = hq // w.G
        kb, vb = synth.bits(p["k"][b, h]), synth.bits(p["v"][b, h])
        ref, ref_lse = orc.window_attention(qb[b, hq:hq + 1], kb, vb, w.L_obs)
        H.check_attention(out[b, hq], out16[b, hq], lse[b, hq], ref.reshape(-1, w.d), ref_lse.reshape(-1),
                          f"cfg4 window b{b} head {hq}")
        ref_sc = orc.scored_range_lse(qb[b, hq:hq + 1], kb, w.L_obs)
        assert np.all(np.abs(lse_sc[b, hq].cpu().double().numpy() - ref_sc.reshape(-1)) <= 1e-3)
