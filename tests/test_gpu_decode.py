"""GPU parity: catekv_append / catekv_decode_plan / catekv_decode_attn against the CPU oracle."""
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


def _run_decode(ck, oc, q_bits, num_ctas, max_new=0, scale=0.0):
    cache = H.device_cache_from_oracle(ck, oc, max_new)
    plan = ck.DecodePlan(cache, num_ctas)
    ck.catekv_decode_plan(cache, plan)
    q = synth.from_bits(q_bits, "cuda")
    B, Hq, d = q.shape
    o32 = torch.full((B, Hq, d), float("nan"), dtype=torch.float32, device="cuda")
    o16 = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    ck.catekv_decode_attn(cache, q, plan, o32, lse, sm_scale=scale)
    ck.catekv_decode_attn(cache, q, plan, o16, None, sm_scale=scale)
    torch.cuda.synchronize()
    return cache, plan, o32, o16, lse


@pytest.mark.parametrize("G", [1, 4, 7, 8])
@pytest.mark.parametrize("num_ctas", [1, 5, 296])
def test_decode_ragged_lengths(ck, G, num_ctas):
    # odd lengths around the 16-row MMA block and the 64-row tile, an empty list, one long list
    lens = [0, 1, 15, 16, 17, 63, 64, 65, 255, 257, 1000, 3]
    B, Hkv = 3, 4
    oc = H.random_cache(B, Hkv, lens, seed=100 + G)
    q = synth.bits(synth.randn_bf16((B, Hkv * G, 128), "cpu", 200 + G, "q"))
    ref, ref_lse = orc.decode_attention(oc, q)
    _, _, o32, o16, lse = _run_decode(ck, oc, q, num_ctas)
    H.check_attention(o32, o16, lse, ref, ref_lse, f"G={G} ctas={num_ctas}")
    # the empty segment gives exact zeros and -inf
    assert torch.all(o32[0, :G] == 0) and torch.all(torch.isinf(lse[0, :G]))
    assert not torch.isnan(o32).any() and not torch.isnan(o16.float()).any()


def test_decode_brute_force_one_head_64_tokens(ck):
    oc = H.random_cache(1, 1, [64], seed=7)
    q = synth.bits(synth.randn_bf16((1, 1, 128), "cpu", 7, "q1"))
    ref, ref_lse = orc.decode_attention(oc, q)
    for ctas in (1, 3):
        _, _, o32, o16, lse = _run_decode(ck, oc, q, ctas)
        H.check_attention(o32, o16, lse, ref, ref_lse)


def test_decode_scale_and_peaked_softmax(ck):
    # a large logit scale makes the softmax one-hot: exercises the running max
    oc = H.random_cache(1, 2, [777, 130], seed=9)
    q = synth.bits(synth.randn_bf16((1, 8, 128), "cpu", 9, "q"))
    for scale in (1.0, 0.01):
        ref, ref_lse = orc.decode_attention(oc, q, scale=scale)
        _, _, o32, o16, lse = _run_decode(ck, oc, q, 11, scale=scale)
        H.check_attention(o32, o16, lse, ref, ref_lse, f"scale={scale}")


def test_decode_split_invariance(ck):
    # the result may not depend on how the rows are cut into CTA ranges (up to fp32 merge rounding)
    lens = [5000, 40, 2048, 911]
    oc = H.random_cache(1, 4, lens, seed=11)
    q = synth.bits(synth.randn_bf16((1, 16, 128), "cpu", 11, "q"))
    outs = [_run_decode(ck, oc, q, n)[2].cpu().double().numpy() for n in (1, 2, 64, 500)]
    for o in outs[1:]:
        assert H.rel_l2(o, outs[0]) < 2e-6


def test_append_then_decode_with_stale_plan(ck):
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=512, B=2)
    lens = [100, 128, 1, 0, 300, 64, 17, 255]
    oc = H.random_cache(2, 4, lens, seed=13)
    cache = H.device_cache_from_oracle(ck, oc, max_new=20)
    plan = ck.DecodePlan(cache, 9)
    ck.catekv_decode_plan(cache, plan)  # built once; the lists then grow under it
    out = torch.empty((2, 16, 128), dtype=torch.float32, device="cuda")
    for step in range(20):
        kn = synth.randn_bf16((2, 4, 128), "cpu", 13, "kn", step)
        vn = synth.randn_bf16((2, 4, 128), "cpu", 13, "vn", step)
        q = synth.randn_bf16((2, 16, 128), "cpu", 13, "q", step)
        ck.catekv_append(cache, kn.cuda(), vn.cuda())
        oc.append(synth.bits(kn), synth.bits(vn))
        ck.catekv_decode_attn(cache, q.cuda(), plan, out)
        if step in (0, 1, 19):
            ref, _ = orc.decode_attention(oc, synth.bits(q))
            H.check_attention(out, None, None, ref, None, f"step {step}")
    torch.cuda.synchronize()
    assert list(cache.seg_len) == [l + 20 for l in lens]
    assert cache.seg_len_dev.cpu().tolist() == [l + 20 for l in lens]
    # pool bytes: the appended rows sit right after the old ones
    for i in range(8):
        o, L = int(cache.seg_off[i]), lens[i] + 20
        assert np.array_equal(synth.bits(cache.k_pool[o:o + L]), oc.k_rows[i])
        assert np.array_equal(synth.bits(cache.v_pool[o:o + L]), oc.v_rows[i])
    # one more append overflows the 128-aligned capacity of some segment: refused, nothing changes
    full = [i for i in range(8) if cache.seg_len[i] == cache.seg_cap[i]]
    if not full:
        while all(cache.seg_len[i] < cache.seg_cap[i] for i in range(8)):
            ck.catekv_append(cache, kn.cuda(), vn.cuda())
    before = cache.seg_len.copy()
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_append(cache, kn.cuda(), vn.cuda())
    assert e.value.code == ck.ERR_CAPACITY
    torch.cuda.synchronize()
    assert np.array_equal(cache.seg_len, before) and cache.seg_len_dev.cpu().tolist() == before.tolist()


@pytest.mark.parametrize("num_ctas", [1, 9, 40])
def test_decode_with_stale_plan_after_segments_shrank(ck, num_ctas):
    """A plan built for longer lists stays valid when lists get shorter (a per-step cache that is refilled with
    fewer rows): rows behind the live length are left out, whole pieces included; a list cut to nothing gives 0."""
    lens = [700, 64, 1500, 3, 90, 400, 2000, 128]
    new_lens = [693, 64, 130, 0, 1, 399, 1999, 17]  # by a few rows, across piece boundaries, to one row, to nothing
    oc = H.random_cache(2, 4, lens, seed=23)
    cache = H.device_cache_from_oracle(ck, oc, max_new=8)
    plan = ck.DecodePlan(cache, num_ctas)
    ck.catekv_decode_plan(cache, plan)
    cache.set_lengths(new_lens)
    short = orc.HybridCache(2, 4, 128)
    for i, L in enumerate(new_lens):
        short.k_rows.append(oc.k_rows[i][:L])
        short.v_rows.append(oc.v_rows[i][:L])
    q = synth.randn_bf16((2, 16, 128), "cpu", 23, "q")
    o32 = torch.full((2, 16, 128), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((2, 16), float("nan"), dtype=torch.float32, device="cuda")
    ck.catekv_decode_attn(cache, q.cuda(), plan, o32, lse)
    torch.cuda.synchronize()
    ref, ref_lse = orc.decode_attention(short, synth.bits(q))
    H.check_attention(o32, None, lse, ref, ref_lse, "shrunk")
    assert torch.all(o32[0, 12:16] == 0)  # the emptied list (sequence 0, KV head 3)
    # the fused append needs lengths that are not below the plan's
    kn = synth.randn_bf16((2, 4, 128), "cuda", 23, "kn")
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_append_decode_attn(cache, kn, kn, q.cuda(), plan, o32, lse)
    assert e.value.code == ck.ERR_INVALID_ARG
    # grown back (and beyond): the same plan again
    cache.set_lengths(lens)
    ck.catekv_decode_attn(cache, q.cuda(), plan, o32, lse)
    torch.cuda.synchronize()
    ref, ref_lse = orc.decode_attention(oc, synth.bits(q))
    H.check_attention(o32, None, lse, ref, ref_lse, "restored")


def test_cache_regrow_lets_full_segments_keep_growing(ck):
    lens = [100, 128, 1, 0, 300, 64, 17, 255]
    oc = H.random_cache(2, 4, lens, seed=29)
    cache = H.device_cache_from_oracle(ck, oc, max_new=0)  # capacities round_up(len, 128): some are full
    kn = synth.randn_bf16((2, 4, 128), "cuda", 29, "kn")
    vn = synth.randn_bf16((2, 4, 128), "cuda", 29, "vn")
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_append(cache, kn, vn)
    assert e.value.code == ck.ERR_CAPACITY
    big = ck.catekv_cache_regrow(cache, max_new=40)
    torch.cuda.synchronize()
    assert list(big.seg_len) == lens == big.seg_len_dev.cpu().tolist()
    for i, L in enumerate(lens):
        o = int(big.seg_off[i])
        assert np.array_equal(synth.bits(big.k_pool[o:o + L]), oc.k_rows[i])
        assert np.array_equal(synth.bits(big.v_pool[o:o + L]), oc.v_rows[i])
    plan = ck.DecodePlan(big, 11)
    ck.catekv_decode_plan(big, plan)
    out = torch.empty((2, 16, 128), dtype=torch.float32, device="cuda")
    for step in range(40):
        kn = synth.randn_bf16((2, 4, 128), "cuda", 29, "kn", step)
        vn = synth.randn_bf16((2, 4, 128), "cuda", 29, "vn", step)
        q = synth.randn_bf16((2, 16, 128), "cuda", 29, "q", step)
        ck.catekv_append_decode_attn(big, kn, vn, q, plan, out)
        oc.append(synth.bits(kn), synth.bits(vn))
    ref, _ = orc.decode_attention(oc, synth.bits(q))
    H.check_attention(out, None, None, ref, None, "after regrow")
    # a destination that is too small, or the cache itself, is refused
    small = ck.Cache(2, 4, [8] * 8, 0, "cuda")
    for dst, code in ((small, ck.ERR_CAPACITY), (big, ck.ERR_INVALID_ARG)):
        rc = ck._lib.catekv_cache_regrow(ck.C.byref(big.struct), ck.C.byref(dst.struct), None)
        assert rc == code


@pytest.mark.parametrize("fused", [False, True])
def test_paged_growth_past_the_laid_out_capacity(ck, fused):
    """Segments outgrow their capacity into overflow pages: appends land there, attention reads base rows and
    pages under plans built before and after the growth, and a regrow gathers everything back."""
    lens = [100, 128, 1, 0, 300, 64, 17, 255]
    B, Hkv, G = 2, 4, 4
    oc = H.random_cache(B, Hkv, lens, seed=31)
    cache = H.device_cache_from_oracle(ck, oc, max_new=0)  # capacities round_up(len, 128): two segments are full
    steps = 150  # up to three pages per segment
    kn = synth.randn_bf16((B, Hkv, 128), "cuda", 31, "kn")
    vn = synth.randn_bf16((B, Hkv, 128), "cuda", 31, "vn")
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_append(cache, kn, vn)
    assert e.value.code == ck.ERR_CAPACITY
    pg = cache.attach_pages(n_pages=24, max_pages=3)
    with pytest.raises(ck.CatekvError) as e:  # pages attached but none handed out yet
        ck.catekv_append(cache, kn, vn)
    assert e.value.code == ck.ERR_CAPACITY
    with pytest.raises(ck.CatekvError) as e:  # more than the pools hold: refused, nothing changed
        ck.catekv_pages_reserve(cache, 64 * 3 + 129)
    assert e.value.code == ck.ERR_CAPACITY and pg.struct.next_free == 0 and not pg.seg_pages.any()
    plan = ck.DecodePlan(cache, 9)
    ck.catekv_decode_plan(cache, plan)  # before any growth
    out = torch.empty((B, Hkv * G, 128), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, Hkv * G), dtype=torch.float32, device="cuda")
    for step in range(steps):
        if step % 50 == 0:
            ck.catekv_pages_reserve(cache, 50)  # in instalments: later pages join the earlier ones
        kn = synth.randn_bf16((B, Hkv, 128), "cuda", 31, "kn", step)
        vn = synth.randn_bf16((B, Hkv, 128), "cuda", 31, "vn", step)
        q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 31, "q", step)
        if fused:
            ck.catekv_append_decode_attn(cache, kn, vn, q, plan, out, lse)
        else:
            ck.catekv_append(cache, kn, vn)
            ck.catekv_decode_attn(cache, q, plan, out, lse)
        oc.append(synth.bits(kn), synth.bits(vn))
        if step in (0, 27, 28, 63, 64, 65, 149):
            ref, ref_lse = orc.decode_attention(oc, synth.bits(q))
            H.check_attention(out, None, lse, ref, ref_lse, f"paged step {step}")
        if step == 90:
            ck.catekv_decode_plan(cache, plan)  # a plan whose plan-time rows lie in pages
    torch.cuda.synchronize()
    assert list(cache.seg_len) == [L + steps for L in lens] == cache.seg_len_dev.cpu().tolist()
    want_pages = [max(0, -(-(L + steps - int(c)) // 64)) for L, c in zip(lens, cache.seg_cap)]
    assert list(pg.seg_pages) == want_pages and pg.struct.next_free == sum(want_pages)
    assert np.array_equal(pg.table_dev.cpu().numpy(), pg.table)
    used = pg.table[pg.table >= 0]
    assert len(set(used.tolist())) == len(used) == sum(want_pages)  # every page handed out once
    # rows: base part in the cache's pools, the rest in the pages of the table
    for i, L0 in enumerate(lens):
        cap, L = int(cache.seg_cap[i]), L0 + steps
        o = int(cache.seg_off[i])
        assert np.array_equal(synth.bits(cache.k_pool[o:o + min(L, cap)]), oc.k_rows[i][:cap])
        for p_i in range(want_pages[i]):
            r0 = cap + 64 * p_i
            nrows = min(64, L - r0)
            page = int(pg.table[i, p_i])
            assert np.array_equal(synth.bits(pg.k_ovf[page * 64:page * 64 + nrows]), oc.k_rows[i][r0:r0 + nrows])
            assert np.array_equal(synth.bits(pg.v_ovf[page * 64:page * 64 + nrows]), oc.v_rows[i][r0:r0 + nrows])
    # the variant with the library's own scratch follows the pages too: same kernel, same bits
    out_a, out_b = torch.empty_like(out), torch.empty_like(out)
    ck.catekv_decode_attn(cache, q, plan, out_a)
    ck.catekv_decode_attn_noalloc(cache, q, plan, out_b)
    torch.cuda.synchronize()
    assert torch.equal(out_a, out_b)
    # the table row of a segment is full: one row more is refused
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_pages_reserve(cache, 64 * 3)
    assert e.value.code == ck.ERR_CAPACITY
    # gather everything back into one contiguous cache
    big = ck.catekv_cache_regrow(cache, max_new=8)
    torch.cuda.synchronize()
    for i, L0 in enumerate(lens):
        o, L = int(big.seg_off[i]), L0 + steps
        assert np.array_equal(synth.bits(big.k_pool[o:o + L]), oc.k_rows[i])
        assert np.array_equal(synth.bits(big.v_pool[o:o + L]), oc.v_rows[i])
    # calls that walk contiguous segments refuse a paged cache
    assert ck._lib.catekv_retrieval_meta_bytes(ck.C.byref(cache.struct), 8) == 0


def test_decode_is_deterministic(ck):
    oc = H.random_cache(2, 4, [700, 64, 1500, 3, 90, 400, 2000, 128], seed=17)
    q = synth.bits(synth.randn_bf16((2, 16, 128), "cpu", 17, "q"))
    a = _run_decode(ck, oc, q, 40)
    b = _run_decode(ck, oc, q, 40)
    assert torch.equal(a[2], b[2]) and torch.equal(a[3], b[3]) and torch.equal(a[4], b[4])


def test_fused_append_decode_matches_oracle_and_two_call_path(ck):
    lens = [100, 128, 1, 0, 300, 64, 17, 255, 63, 2000, 0, 5]
    oc = H.random_cache(3, 4, lens, seed=19)
    cache = H.device_cache_from_oracle(ck, oc, max_new=24)
    ref_cache = H.device_cache_from_oracle(ck, oc, max_new=24)
    plan = ck.DecodePlan(cache, 13)
    ck.catekv_decode_plan(cache, plan)
    plan2 = ck.DecodePlan(ref_cache, 13)
    ck.catekv_decode_plan(ref_cache, plan2)
    out = torch.empty((3, 28, 128), dtype=torch.float32, device="cuda")
    out2 = torch.empty_like(out)
    lse = torch.empty((3, 28), dtype=torch.float32, device="cuda")
    for step in range(24):
        kn = synth.randn_bf16((3, 4, 128), "cuda", 19, "kn", step)
        vn = synth.randn_bf16((3, 4, 128), "cuda", 19, "vn", step)
        q = synth.randn_bf16((3, 28, 128), "cuda", 19, "q", step)
        ck.catekv_append_decode_attn(cache, kn, vn, q, plan, out, lse)
        ck.catekv_append(ref_cache, kn, vn)
        ck.catekv_decode_attn(ref_cache, q, plan2, out2)
        oc.append(synth.bits(kn), synth.bits(vn))
        assert torch.equal(out, out2), step  # same kernel, same arithmetic
        if step in (0, 1, 23):
            ref, ref_lse = orc.decode_attention(oc, synth.bits(q))
            H.check_attention(out, None, lse, ref, ref_lse, f"fused step {step}")
    torch.cuda.synchronize()
    assert list(cache.seg_len) == [l + 24 for l in lens]
    assert cache.seg_len_dev.cpu().tolist() == [l + 24 for l in lens]
    for i in range(12):
        o, L = int(cache.seg_off[i]), lens[i] + 24
        assert np.array_equal(synth.bits(cache.k_pool[o:o + L]), oc.k_rows[i])
        assert np.array_equal(synth.bits(cache.v_pool[o:o + L]), oc.v_rows[i])
    # a full segment refuses the fused call too, before anything is launched
    while all(cache.seg_len[i] < cache.seg_cap[i] for i in range(12)):
        ck.catekv_append(cache, kn, vn)
    before = cache.seg_len.copy()
    out.fill_(7.0)
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_append_decode_attn(cache, kn, vn, q, plan, out)
    assert e.value.code == ck.ERR_CAPACITY
    torch.cuda.synchronize()
    assert np.array_equal(cache.seg_len, before) and torch.all(out == 7.0)
