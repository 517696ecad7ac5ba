"""GPU parity: query-aware retrieval on adaptive heads (metadata, chunk selection, gathered attention)."""
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


def _meta_of(ck, cache, meta, cs, seg, n_chunks):
    c0 = int(cache.seg_off[seg]) // cs
    m = synth.bits(meta.view(torch.bfloat16).view(-1, 2, 128)[c0:c0 + n_chunks])
    return orc.bf16_to_f64(m[:, 0]), orc.bf16_to_f64(m[:, 1])


_check_selection = H.check_retrieval_band


@pytest.mark.parametrize("cs,G", [(8, 4), (8, 7), (16, 1), (1, 2)])
def test_retrieval_matches_oracle(ck, cs, G):
    lens = [700, 64, 2049, 5, 1300, 0]
    B, Hkv = 2, 3
    oc = H.random_cache(B, Hkv, lens, seed=70 + cs)
    cache = H.device_cache_from_oracle(ck, oc, max_new=8)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    torch.cuda.synchronize()
    # metadata: bit-exact element-wise extremes
    for s, L in enumerate(lens):
        if L:
            kmax, kmin = orc.retrieval_metadata(oc.k_rows[s], cs)
            gmax, gmin = _meta_of(ck, cache, meta, cs, s, kmax.shape[0])
            assert np.array_equal(gmax, kmax) and np.array_equal(gmin, kmin), s
    q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 71, "q", cs)
    qb = orc.bf16_to_f64(synth.bits(q))
    mask = np.array([1, 1, 1, 1, 0, 1], dtype=np.uint8)
    budget, sink, local = 256, 4, 32
    want_len = []
    for s, L in enumerate(lens):
        if mask[s] and L > budget:
            want_len.append(len(orc.retrieve_indices(np.zeros((L + cs - 1) // cs), L, sink, local, budget, cs)))
        else:
            want_len.append(L)
    step = ck.Cache(B, Hkv, want_len, 0, "cuda")
    idx = torch.full((B * Hkv, max(lens)), -1, dtype=torch.int32, device="cuda")
    ck.catekv_retrieve_compact(cache, meta, cs, q, mask, budget, sink, local, step, idx_out=idx)
    torch.cuda.synchronize()
    assert list(step.seg_len) == want_len and step.seg_len_dev.cpu().tolist() == want_len
    idx = idx.cpu().numpy()
    soc = orc.HybridCache(B, Hkv, 128)
    for s, L in enumerate(lens):
        got = idx[s, :want_len[s]].astype(np.int64)
        if mask[s] and L > budget:
            kmax, kmin = orc.retrieval_metadata(oc.k_rows[s], cs)
            b, h = divmod(s, Hkv)
            scores = orc.retrieval_scores(qb[b, h * G:(h + 1) * G], kmax, kmin)
            _check_selection(got, scores, L, sink, local, budget, cs, f"seg {s}")
        else:
            assert np.array_equal(got, np.arange(L))
        o = int(step.seg_off[s])
        assert np.array_equal(synth.bits(step.k_pool[o:o + want_len[s]]), oc.k_rows[s][got])
        assert np.array_equal(synth.bits(step.v_pool[o:o + want_len[s]]), oc.v_rows[s][got])
        soc.k_rows.append(oc.k_rows[s][got])
        soc.v_rows.append(oc.v_rows[s][got])
    # attention over the step cache == oracle attention over the retrieved rows
    plan = ck.DecodePlan(step, 12)
    ck.catekv_decode_plan(step, plan)
    out = torch.empty((B, Hkv * G, 128), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, Hkv * G), dtype=torch.float32, device="cuda")
    ck.catekv_decode_attn(step, q, plan, out, lse)
    ref, ref_lse = orc.decode_attention(soc, synth.bits(q))
    H.check_attention(out, None, lse, ref, ref_lse, f"cs={cs} G={G}")


@pytest.mark.parametrize("one_launch", [False, True])
def test_retrieval_metadata_follows_appends(ck, one_launch):
    cs = 8
    lens = [100, 7, 0, 64]
    oc = H.random_cache(1, 4, lens, seed=75)
    cache = H.device_cache_from_oracle(ck, oc, max_new=20)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    for step in range(20):
        kn = synth.randn_bf16((1, 4, 128), "cuda", 75, "kn", step)
        vn = synth.randn_bf16((1, 4, 128), "cuda", 75, "vn", step)
        if one_launch:
            ck.catekv_append_retrieval(cache, kn, vn, cs, meta)
        else:
            ck.catekv_append(cache, kn, vn)
            ck.catekv_retrieval_append(cache, cs, kn, meta)
        oc.append(synth.bits(kn), synth.bits(vn))
    torch.cuda.synchronize()
    assert list(cache.seg_len) == [L + 20 for L in lens] == cache.seg_len_dev.cpu().tolist()
    for s in range(4):
        o, L = int(cache.seg_off[s]), lens[s] + 20
        assert np.array_equal(synth.bits(cache.k_pool[o:o + L]), oc.k_rows[s])
        assert np.array_equal(synth.bits(cache.v_pool[o:o + L]), oc.v_rows[s])
    for s in range(4):
        kmax, kmin = orc.retrieval_metadata(oc.k_rows[s], cs)
        gmax, gmin = _meta_of(ck, cache, meta, cs, s, kmax.shape[0])
        assert np.array_equal(gmax, kmax) and np.array_equal(gmin, kmin), s


def test_retrieval_finds_loud_keys_and_budget_covers_all(ck):
    # quiet keys plus a few loud ones on the direction the queries lean on: all loud rows are retrieved
    rng = np.random.default_rng(76)
    n, G = 4096, 4
    c = rng.standard_normal(128)
    c /= np.linalg.norm(c)
    K = 0.05 * rng.standard_normal((n, 128))
    loud = np.sort(rng.choice(np.arange(16, n - 80), 12, replace=False))
    K[loud] += 3.0 * c
    oc = orc.HybridCache(1, 1, 128)
    oc.k_rows.append(orc.f64_to_bf16(K))
    oc.v_rows.append(orc.f64_to_bf16(rng.standard_normal((n, 128))))
    cache = H.device_cache_from_oracle(ck, oc, 0)
    meta = ck.catekv_retrieval_meta(cache, 8)
    ck.catekv_retrieval_build(cache, 8, meta)
    q = synth.from_bits(orc.f64_to_bf16(0.1 * rng.standard_normal((1, G, 128)) + 3.0 * c), "cuda")
    step = ck.Cache(1, 1, [n], 0, "cuda")
    idx = torch.full((1, n), -1, dtype=torch.int32, device="cuda")
    ck.catekv_retrieve_compact(cache, meta, 8, q, [1], 256, 4, 64, step, idx_out=idx)
    torch.cuda.synchronize()
    got = idx[0, :int(step.seg_len[0])].cpu().numpy()
    assert len(got) == 256 and set(loud.tolist()) <= set(got.tolist())
    # a budget at or above the length takes every row, as does an unmasked segment
    for mask, budget in (([1], n), ([0], 64)):
        ck.catekv_retrieve_compact(cache, meta, 8, q, mask, budget, 4, 64, step, idx_out=idx)
        torch.cuda.synchronize()
        assert int(step.seg_len[0]) == n and torch.equal(idx[0].cpu(), torch.arange(n, dtype=torch.int32))
    # a step cache that is too small is refused before anything runs
    small = ck.Cache(1, 1, [128], 0, "cuda")
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_retrieve_compact(cache, meta, 8, q, [1], 256, 4, 64, small)
    assert e.value.code == ck.ERR_CAPACITY


@pytest.mark.parametrize("indexed", [False, True])
def test_retrieval_step_replayed_as_cuda_graph(ck, indexed):
    """append + metadata append + retrieve + attention captured once and replayed while the lists grow: the kept
    lengths move within a chunk under a decode plan that was built once, and every step matches the oracle."""
    cs, G, B, Hkv = 8, 4, 2, 2
    lens = [900, 300, 1500, 40]
    budget, sink, local = 256, 4, 32
    steps = 11  # crosses a chunk boundary of every list
    oc = H.random_cache(B, Hkv, lens, seed=81)
    cache = H.device_cache_from_oracle(ck, oc, max_new=steps + 2)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    mask = np.array([1, 1, 1, 0], dtype=np.uint8)
    step_cache = ck.Cache(B, Hkv, [budget + 2 * cs if mask[s] and L > budget else L + steps + 2
                                   for s, L in enumerate(lens)], 0, "cuda")
    q = torch.empty((B, Hkv * G, 128), dtype=torch.bfloat16, device="cuda")
    kn = torch.empty((B, Hkv, 128), dtype=torch.bfloat16, device="cuda")
    vn = torch.empty_like(kn)
    out = torch.empty((B, Hkv * G, 128), dtype=torch.float32, device="cuda")
    idx = torch.full((B * Hkv, max(lens) + steps + 2), -1, dtype=torch.int32, device="cuda")
    ws = ck.retrieve_workspace(cache)
    sel = torch.full((B * Hkv,), -99, dtype=torch.int32, device="cuda")
    if indexed:
        view = ck.CacheView(cache, ck.catekv_retrieve_lengths(cache, cs, mask, budget, sink, local))
        plan = ck.DecodePlan(view, 7)
        ck.catekv_decode_plan(view, plan)  # once, from the lengths before the first step
    else:
        ck.catekv_retrieve_compact(cache, meta, cs, q.zero_(), mask, budget, sink, local, step_cache, ws=ws)
        plan = ck.DecodePlan(step_cache, 7)
        ck.catekv_decode_plan(step_cache, plan)  # once, from the lengths of this first fill

    def one_step():
        if indexed:  # the one-launch form of the two appends
            ck.catekv_append_retrieval(cache, kn, vn, cs, meta)
        else:
            ck.catekv_append(cache, kn, vn)
            ck.catekv_retrieval_append(cache, cs, kn, meta)
        if indexed:
            ck.catekv_retrieve_select(cache, meta, cs, q, mask, budget, sink, local, idx, sel, ws=ws)
            ck.catekv_decode_attn_indexed(cache, idx, sel, q, plan, out)
        else:
            ck.catekv_retrieve_compact(cache, meta, cs, q, mask, budget, sink, local, step_cache, idx_out=idx, ws=ws)
            ck.catekv_decode_attn(step_cache, q, plan, out)

    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            one_step()  # host code only: the host mirror of `cache` advances by one row
    torch.cuda.current_stream().wait_stream(side)
    seen_lens = set()
    for t in range(steps):
        q.copy_(synth.randn_bf16((B, Hkv * G, 128), "cuda", 81, "q", t))
        kn.copy_(synth.randn_bf16((B, Hkv, 128), "cuda", 81, "kn", t))
        vn.copy_(synth.randn_bf16((B, Hkv, 128), "cuda", 81, "vn", t))
        if t:
            ck.catekv_cache_advance(cache, 1)
        g.replay()
        torch.cuda.synchronize()
        oc.append(synth.bits(kn), synth.bits(vn))
        qb = orc.bf16_to_f64(synth.bits(q))
        got_len = sel.cpu().tolist() if indexed else step_cache.seg_len_dev.cpu().tolist()
        got_idx = idx.cpu().numpy()
        soc = orc.HybridCache(B, Hkv, 128)
        for s in range(B * Hkv):
            L = lens[s] + t + 1
            if indexed and not (mask[s] and L > budget):
                assert got_len[s] == -1
                got = np.arange(L)
            else:
                got = got_idx[s, :got_len[s]].astype(np.int64)
            if mask[s] and L > budget:
                kmax, kmin = orc.retrieval_metadata(oc.k_rows[s], cs)
                b, h = divmod(s, Hkv)
                scores = orc.retrieval_scores(qb[b, h * G:(h + 1) * G], kmax, kmin)
                _check_selection(got, scores, L, sink, local, budget, cs, f"step {t} seg {s}")
            else:
                assert np.array_equal(got, np.arange(L)), (t, s)
            soc.k_rows.append(oc.k_rows[s][got])
            soc.v_rows.append(oc.v_rows[s][got])
        seen_lens.add(got_len[0])
        ref, _ = orc.decode_attention(soc, synth.bits(q))
        H.check_attention(out, None, None, ref, None, f"graph step {t}")
    assert len(seen_lens) > 1  # the kept length did move under the plan
    assert list(cache.seg_len) == [L + steps for L in lens] == cache.seg_len_dev.cpu().tolist()


@pytest.mark.parametrize("cs,G,num_ctas", [(8, 4, 12), (8, 7, 296), (16, 1, 3), (1, 2, 12)])
def test_retrieve_select_and_indexed_attention(ck, cs, G, num_ctas):
    """Retrieval without the copy: index lists + attention in place == oracle == the gather path bit for bit."""
    lens = [700, 64, 2049, 5, 1300, 0]
    B, Hkv = 2, 3
    oc = H.random_cache(B, Hkv, lens, seed=90 + cs)
    cache = H.device_cache_from_oracle(ck, oc, max_new=8)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 91, "q", cs)
    qb = orc.bf16_to_f64(synth.bits(q))
    mask = np.array([1, 1, 1, 1, 0, 1], dtype=np.uint8)
    budget, sink, local = 256, 4, 32
    want = ck.catekv_retrieve_lengths(cache, cs, mask, budget, sink, local)
    for s, L in enumerate(lens):
        if mask[s] and L > budget:
            assert want[s] == len(orc.retrieve_indices(np.zeros((L + cs - 1) // cs), L, sink, local, budget, cs))
        else:
            assert want[s] == L
    idx = torch.full((B * Hkv, int(want.max()) + 3), -7, dtype=torch.int32, device="cuda")
    sel = torch.full((B * Hkv,), -99, dtype=torch.int32, device="cuda")
    ck.catekv_retrieve_select(cache, meta, cs, q, mask, budget, sink, local, idx, sel)
    torch.cuda.synchronize()
    got_sel = sel.cpu().tolist()
    soc = orc.HybridCache(B, Hkv, 128)
    for s, L in enumerate(lens):
        if mask[s] and L > budget:
            assert got_sel[s] == want[s]
            got = idx[s, :want[s]].cpu().numpy().astype(np.int64)
            kmax, kmin = orc.retrieval_metadata(oc.k_rows[s], cs)
            b, h = divmod(s, Hkv)
            scores = orc.retrieval_scores(qb[b, h * G:(h + 1) * G], kmax, kmin)
            _check_selection(got, scores, L, sink, local, budget, cs, f"seg {s}")
            assert torch.all(idx[s, want[s]:] == -7)  # nothing written behind the list
        else:
            assert got_sel[s] == -1 and torch.all(idx[s] == -7)
            got = np.arange(L)
        soc.k_rows.append(oc.k_rows[s][got])
        soc.v_rows.append(oc.v_rows[s][got])
    view = ck.CacheView(cache, want)
    plan = ck.DecodePlan(view, num_ctas)
    ck.catekv_decode_plan(view, plan)
    out = torch.full((B, Hkv * G, 128), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B, Hkv * G), float("nan"), dtype=torch.float32, device="cuda")
    ck.catekv_decode_attn_indexed(cache, idx, sel, q, plan, out, lse)
    o16 = torch.full((B, Hkv * G, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    ck.catekv_decode_attn_indexed(cache, idx, sel, q, plan, o16)
    ref, ref_lse = orc.decode_attention(soc, synth.bits(q))
    H.check_attention(out, o16, lse, ref, ref_lse, f"indexed cs={cs} G={G}")
    # the gather path attends to the same rows in the same order under the same split: identical bits
    step = ck.Cache(B, Hkv, want, 0, "cuda")
    ck.catekv_retrieve_compact(cache, meta, cs, q, mask, budget, sink, local, step)
    plan2 = ck.DecodePlan(step, num_ctas)
    ck.catekv_decode_plan(step, plan2)
    out2 = torch.empty_like(out)
    lse2 = torch.empty_like(lse)
    ck.catekv_decode_attn(step, q, plan2, out2, lse2)
    torch.cuda.synchronize()
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    # an index row that is too short for a kept list is refused before anything runs
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_retrieve_select(cache, meta, cs, q, mask, budget, sink, local, idx[:, :100].contiguous(), sel)
    assert e.value.code == ck.ERR_INVALID_ARG


def _one_dim_case(ck, levels, budget, cs=8, sink=4, local=32):
    """One segment whose keys live on dimension 0 only and a query that is 1 there: the bound of a chunk is the
    largest of its keys' values, exact on both sides, so the selection must equal the oracle's list (ties to the
    lowest chunk) and not just agree within the band."""
    n = len(levels)
    K = np.zeros((n, 128))
    K[:, 0] = levels
    oc = orc.HybridCache(1, 1, 128)
    oc.k_rows.append(orc.f64_to_bf16(K))
    oc.v_rows.append(orc.f64_to_bf16(np.zeros((n, 128))))
    assert np.array_equal(orc.bf16_to_f64(oc.k_rows[0])[:, 0], levels)  # the levels are bf16 values
    cache = H.device_cache_from_oracle(ck, oc, 0)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    qv = np.zeros((1, 2, 128))
    qv[:, :, 0] = 1.0
    q = synth.from_bits(orc.f64_to_bf16(qv), "cuda")
    kmax, kmin = orc.retrieval_metadata(oc.k_rows[0], cs)
    scores = orc.retrieval_scores(qv[0], kmax, kmin)
    want = orc.retrieve_indices(scores, n, sink, local, budget, cs)
    idx = torch.full((1, len(want) + 8), -7, dtype=torch.int32, device="cuda")
    sel = torch.full((1,), -99, dtype=torch.int32, device="cuda")
    ck.catekv_retrieve_select(cache, meta, cs, q, [1], budget, sink, local, idx, sel)
    torch.cuda.synchronize()
    if int(sel[0]) == -1:  # the whole list
        assert np.array_equal(want, np.arange(n)) and torch.all(idx[0] == -7)
        return
    assert int(sel[0]) == len(want)
    assert np.array_equal(idx[0, :len(want)].cpu().numpy().astype(np.int64), want)
    assert torch.all(idx[0, len(want):] == -7)


@pytest.mark.parametrize("case", ["three_levels", "all_equal", "outlier", "two_neighbours", "negative", "random"])
@pytest.mark.parametrize("n,budget", [(8192 + 40, 1024), (3000, 520), (20000, 2048), (230000, 4096)])
def test_retrieval_selection_with_ties_and_crowded_scores(ck, case, n, budget):
    """The short-list selection kernel on score distributions that stress each of its steps: hundreds of exact
    ties at the threshold, one score for all, an outlier that squeezes every other score into one histogram bin,
    two adjacent bf16 values, negative scores, and plain random ones."""
    rng = np.random.default_rng(len(case) * 1000 + n)
    chunk_level = {
        "three_levels": lambda c: rng.integers(1, 4, c).astype(np.float64),
        "all_equal": lambda c: np.full(c, 1.5),
        "outlier": lambda c: np.concatenate([[4096.0], rng.integers(0, 256, c - 1) / 256.0]),
        "two_neighbours": lambda c: np.where(rng.random(c) < 0.5, 2.0, 2.015625),
        "negative": lambda c: -rng.integers(1, 200, c) / 16.0,
        "random": lambda c: orc.bf16_to_f64(orc.f64_to_bf16(rng.standard_normal(c))),
    }[case]
    n_chunks = (n + 7) // 8
    lv = chunk_level(n_chunks)
    if case == "outlier":
        lv = np.roll(lv, n_chunks // 2)
    levels = np.repeat(lv, 8)[:n]
    _one_dim_case(ck, levels, budget)


def test_retrieval_many_short_segments(ck):
    """A thousand segments of one to three metadata tiles each: a CTA of the scoring kernel walks across several
    segments (masked out, too short to select, and empty ones among them); every selection is checked."""
    rng = np.random.default_rng(97)
    B, Hkv, G, cs = 125, 8, 2, 8
    budget, sink, local = 200, 4, 16
    lens = rng.integers(300, 1400, B * Hkv)
    lens[rng.random(B * Hkv) < 0.1] = 0
    lens[rng.random(B * Hkv) < 0.1] = 150          # not longer than the budget: kept whole
    mask = (rng.random(B * Hkv) < 0.8).astype(np.uint8)
    oc = H.random_cache(B, Hkv, lens.tolist(), seed=97)
    cache = H.device_cache_from_oracle(ck, oc, max_new=8)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 97, "q")
    qb = orc.bf16_to_f64(synth.bits(q))
    want = ck.catekv_retrieve_lengths(cache, cs, mask, budget, sink, local)
    idx = torch.full((B * Hkv, int(want.max()) + 3), -7, dtype=torch.int32, device="cuda")
    sel = torch.full((B * Hkv,), -99, dtype=torch.int32, device="cuda")
    ck.catekv_retrieve_select(cache, meta, cs, q, mask, budget, sink, local, idx, sel)
    torch.cuda.synchronize()
    got_sel = sel.cpu().tolist()
    idx = idx.cpu().numpy()
    n_selecting = 0
    for s, L in enumerate(lens.tolist()):
        if mask[s] and L > budget:
            n_selecting += 1
            assert got_sel[s] == want[s], s
            kmax, kmin = orc.retrieval_metadata(oc.k_rows[s], cs)
            b, h = divmod(s, Hkv)
            scores = orc.retrieval_scores(qb[b, h * G:(h + 1) * G], kmax, kmin)
            _check_selection(idx[s, :want[s]].astype(np.int64), scores, L, sink, local, budget, cs, f"seg {s}")
            assert np.all(idx[s, want[s]:] == -7)
        else:
            assert got_sel[s] == -1 and np.all(idx[s] == -7), s
    assert n_selecting > 500


def test_retrieval_selection_random_exact_cases(ck):
    """Seeded sweep over chunk sizes, lengths, budgets, sink / local sizes and score distributions (few levels, one
    value, an outlier, two adjacent bf16 values, negative, normal, heavy-tailed with both signs), every case with
    scores that are exact on both sides: the device's list must equal the oracle's."""
    rng = np.random.default_rng(2024)
    for it in range(60):
        cs = int(rng.choice([1, 2, 4, 8, 16]))
        n = int(rng.integers(50, 40000)) if cs >= 4 else int(rng.integers(50, 12000))
        sink, local = int(rng.integers(0, 20)), int(rng.integers(0, 100))
        budget = int(rng.integers(8, max(9, n)))
        nch = (n + cs - 1) // cs
        kind = it % 7
        if kind == 0:
            lv = rng.integers(1, 4, nch).astype(np.float64)
        elif kind == 1:
            lv = np.full(nch, 0.75)
        elif kind == 2:
            lv = np.roll(np.concatenate([[4096.0], rng.integers(0, 256, nch - 1) / 256.0]), int(rng.integers(0, nch)))
        elif kind == 3:
            lv = np.where(rng.random(nch) < 0.5, 2.0, 2.015625)
        elif kind == 4:
            lv = -rng.integers(1, 200, nch) / 16.0
        elif kind == 5:
            lv = orc.bf16_to_f64(orc.f64_to_bf16(rng.standard_normal(nch)))
        else:
            lv = orc.bf16_to_f64(orc.f64_to_bf16(np.exp(3 * rng.standard_normal(nch)) * rng.choice([-1, 1], nch)))
        _one_dim_case(ck, np.repeat(lv, cs)[:n], budget, cs=cs, sink=sink, local=local)
