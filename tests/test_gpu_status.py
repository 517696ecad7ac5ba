"""GPU: how a kernel-side failure reaches the host.  Nothing here faults or hangs: a bounded wait is made to run
out with nothing in flight, a copy is cut at its destination's capacity, and the status block says so."""
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


def test_status_block_is_read_reported_and_cleared(ck):
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    assert ck.catekv_workspace_status(ws) == {"flags": 0, "kernel": 0, "segment": 0, "index": 0}
    # a block that a kernel has written (set here by a plain copy): the call returns the device-error code
    ws[:16].view(torch.int32).copy_(torch.tensor([ck.STATUS_CAPACITY, 3, 5, 129], dtype=torch.int32))
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_workspace_status(ws)
    assert e.value.code == ck.ERR_DEVICE
    st = ck.catekv_workspace_status(ws, clear=True, raise_on_error=False)
    assert st == {"flags": ck.STATUS_CAPACITY, "kernel": 3, "segment": 5, "index": 129}
    assert ck.catekv_workspace_status(ws)["flags"] == 0  # cleared by the read before


def _select_inputs():
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=2048, budget=160)
    p = synth.prefill_layer(w, 0)
    return w, p, p["head_mask"]


def test_expired_scoring_waits_are_reported_and_the_next_call_is_clean(ck):
    w, p, mask = _select_inputs()
    lens = [w.budget if mask[0, h] else w.n for h in range(w.Hkv)]
    cache = ck.Cache(w.B, w.Hkv, lens, 0, "cuda")
    ws = torch.empty(ck.catekv_select_workspace_bytes(w.B, w.Hq, w.Hkv, w.n, w.L_obs), dtype=torch.uint8, device="cuda")
    args = (p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda(), p["seq_len"], mask, cache, w.budget, w.eta, w.sink, w.local,
            w.pool_mode, w.pool_param)
    # both scoring passes of this call run with an idle producer lane: every wait runs out, nothing is in flight
    ck.catekv_test_expire_score_waits(2)
    ck.catekv_select_compact(*args, ws=ws)
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_workspace_status(ws)
    assert e.value.code == ck.ERR_DEVICE
    st = ck.catekv_workspace_status(ws, raise_on_error=False)
    assert st["flags"] & ck.STATUS_WAIT_EXPIRED and st["kernel"] == 1
    # the context is intact; the same workspace serves a healthy call whose result matches the oracle
    idx = torch.full((w.B * w.Hkv, w.n), -1, dtype=torch.int32, device="cuda")
    ck.catekv_select_compact(*args, ws=ws, idx_out=idx)
    assert ck.catekv_workspace_status(ws)["flags"] == 0
    qw, k = synth.bits(p["q_win"]), synth.bits(p["k"])
    for h in range(w.Hkv):
        if mask[0, h]:
            C = orc.window_scores(qw[0, h * w.G:(h + 1) * w.G], k[0, h], w.L_obs)
            got = idx[h, :int(cache.seg_len[h])].cpu().numpy()
            H.check_indices_band(got, C, w.n, w.sink, w.local, w.budget, w.pool_mode, w.pool_param, f"h{h}")


def test_expired_waits_in_head_cv_are_reported(ck):
    wq = synth.scaled(synth.WORKLOADS["cfg4"], L_obs=32)
    types = np.array([1, 0, 1, 0], dtype=np.uint8)
    q, k = synth.calibration_prompt(wq, 0, 0, 2048, types)
    ws = torch.empty(ck.catekv_head_cv_workspace_bytes(1, wq.Hq, wq.Hkv, 2048, 32, 64, 32), dtype=torch.uint8, device="cuda")
    ck.catekv_test_expire_score_waits(1)  # the first pass only: the second then runs on statistics that never came
    ck.catekv_head_cv(q.cuda(), k.cuda(), [2048], 64, 32, 0.99, 1.0, True, ws=ws)
    st = ck.catekv_workspace_status(ws, raise_on_error=False)
    assert st["flags"] & ck.STATUS_WAIT_EXPIRED
    cv = ck.catekv_head_cv(q.cuda(), k.cuda(), [2048], 64, 32, 0.99, 1.0, True, ws=ws).cpu().numpy()
    assert ck.catekv_workspace_status(ws)["flags"] == 0
    ref = orc.head_cv(synth.bits(q), synth.bits(k), [2048], 32, 64, 32, float(np.float32(0.99)), 1.0, True)
    np.testing.assert_allclose(cv, ref, rtol=1e-3)


def test_expired_waits_in_window_attention_are_reported(ck):
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=1500)
    p = synth.prefill_layer(w, 0)
    qw, k, v = p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda()
    ws = torch.empty(ck._lib.catekv_window_attn_workspace_bytes(w.B, w.Hq, w.Hkv, w.n, w.L_obs), dtype=torch.uint8,
                     device="cuda")
    ck.catekv_test_expire_score_waits(1)
    ck.catekv_window_attn(qw, k, v, [w.n], ws=ws)
    st = ck.catekv_workspace_status(ws, raise_on_error=False)
    assert st["flags"] & ck.STATUS_WAIT_EXPIRED
    out, lse, _ = ck.catekv_window_attn(qw, k, v, [w.n], ws=ws)   # same workspace, healthy call
    assert ck.catekv_workspace_status(ws)["flags"] == 0
    ref, ref_lse = orc.window_attention(synth.bits(p["q_win"])[0, :w.G], synth.bits(p["k"])[0, 0], synth.bits(p["v"])[0, 0],
                                        w.L_obs)
    H.check_attention(out[0, :w.G].reshape(-1, w.d), None, lse[0, :w.G].reshape(-1), ref.reshape(-1, w.d),
                      ref_lse.reshape(-1), "after an expired call")


def test_replayed_gather_is_cut_at_the_step_cache_capacity(ck):
    """A retrieval step captured once and replayed while the source grows past what the step cache can hold: the
    copy stops at the capacity, nothing behind the segment is written, and the status block reports it."""
    cs, G, B, Hkv = 8, 4, 1, 2
    lens = [300, 120]           # segment 1 is copied whole (mask 0); its step segment holds 128 rows
    budget, sink, local = 64, 4, 16
    steps = 12                  # 120 + 12 = 132 > 128
    oc = H.random_cache(B, Hkv, lens, seed=91)
    cache = H.device_cache_from_oracle(ck, oc, max_new=steps + 4)
    meta = ck.catekv_retrieval_meta(cache, cs)
    ck.catekv_retrieval_build(cache, cs, meta)
    mask = np.array([1, 0], dtype=np.uint8)
    # the step cache: a roomy first segment (so that the gather's grid spans 512 rows) and a tight last one; its
    # pools get a margin of 128 rows behind the last segment, filled with a sentinel, where an unclamped copy would land
    step_cache = ck.Cache(B, Hkv, [400, 121], 0, "cuda")
    assert list(step_cache.seg_cap) == [512, 128] and step_cache.total_rows == 640
    sentinel = 0x7B7B
    step_cache.k_pool = torch.full((768, 128), 0, dtype=torch.int16, device="cuda").fill_(sentinel).view(torch.bfloat16)
    step_cache.v_pool = torch.full((768, 128), 0, dtype=torch.int16, device="cuda").fill_(sentinel).view(torch.bfloat16)
    step_cache.struct.k_pool = step_cache.k_pool.data_ptr()
    step_cache.struct.v_pool = step_cache.v_pool.data_ptr()
    q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 91, "q")
    kn = synth.randn_bf16((B, Hkv, 128), "cuda", 91, "kn")
    vn = synth.randn_bf16((B, Hkv, 128), "cuda", 91, "vn")
    ws = ck.retrieve_workspace(cache)

    def one_step():
        ck.catekv_append_retrieval(cache, kn, vn, cs, meta)
        ck.catekv_retrieve_compact(cache, meta, cs, q, mask, budget, sink, local, step_cache, ws=ws)

    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            one_step()
    torch.cuda.current_stream().wait_stream(side)
    for t in range(steps):
        if t:
            ck.catekv_cache_advance(cache, 1)
        g.replay()
        torch.cuda.synchronize()
        assert int(step_cache.seg_len_dev[1]) == min(lens[1] + t + 1, 128)
        st = ck.catekv_workspace_status(ws, raise_on_error=False)
        assert bool(st["flags"] & ck.STATUS_CAPACITY) == (lens[1] + t + 1 > 128), (t, st)
        if st["flags"]:
            assert st["kernel"] == 3 and st["segment"] == 1
    # nothing was written behind the last segment, and it holds exactly the first 128 rows of its source
    assert torch.all(step_cache.k_pool.view(torch.int16)[640:] == sentinel)
    assert torch.all(step_cache.v_pool.view(torch.int16)[640:] == sentinel)
    src1 = int(cache.seg_off[1])
    assert torch.equal(step_cache.k_pool[512:640], cache.k_pool[src1:src1 + 128])
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_workspace_status(ws, clear=True)
    assert e.value.code == ck.ERR_DEVICE
    assert ck.catekv_workspace_status(ws)["flags"] == 0


def test_chunk_mode_leaves_upper_bounds_until_synced(ck):
    # candidates (n - Lc - S) not a multiple of cs: whether the short last chunk is kept depends on the scores
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=1531, budget=200)
    p = synth.prefill_layer(w, 0)
    mask = p["head_mask"]
    assert (w.n - w.local - w.sink) % 8 != 0
    lens = [w.budget if mask[0, h] else w.n for h in range(w.Hkv)]
    cache = ck.Cache(w.B, w.Hkv, lens, 4, "cuda")
    ck.catekv_select_compact(p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda(), p["seq_len"], mask, cache, w.budget, w.eta,
                             w.sink, w.local, orc.POOL_CHUNK, 8)
    assert cache.struct.reserved == 1
    bound = cache.seg_len.copy()
    # plans and plain attention take the upper bounds; the fused append, which places a row by the plan, refuses
    plan = ck.DecodePlan(cache, 8)
    ck.catekv_decode_plan(cache, plan)
    q, kn, vn = synth.decode_inputs(w, 0, 0, "cuda", mask)
    out = torch.empty((w.B, w.Hq, w.d), dtype=torch.float32, device="cuda")
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_append_decode_attn(cache, kn, vn, q, plan, out)
    assert e.value.code == ck.ERR_INVALID_ARG
    ck.catekv_decode_attn(cache, q, plan, out)
    ck.catekv_cache_sync_lengths(cache)
    assert cache.struct.reserved == 0
    dev = cache.seg_len_dev.cpu().numpy()
    assert np.array_equal(dev, cache.seg_len) and np.all(dev <= bound) and np.all(bound - dev < 8)
    # attention under the upper-bound plan saw exactly the device's rows
    oc = orc.HybridCache(w.B, w.Hkv, w.d)
    for h in range(w.Hkv):
        o, L = int(cache.seg_off[h]), int(dev[h])
        oc.k_rows.append(synth.bits(cache.k_pool[o:o + L]))
        oc.v_rows.append(synth.bits(cache.v_pool[o:o + L]))
    ref, _ = orc.decode_attention(oc, synth.bits(q))
    H.check_attention(out, None, None, ref, None, "upper-bound plan")
    ck.catekv_decode_plan(cache, plan)                          # from the exact lengths
    ck.catekv_append_decode_attn(cache, kn, vn, q, plan, out)  # accepted now


@pytest.mark.trips_checks
def test_checked_build_clamps_a_row_list_that_leaves_its_segment(ck):
    """Checked build only: an index list whose entries point outside the segment (but inside the pool, so that even
    an unchecked library would read legal memory) is clamped into the segment and reported."""
    if not ck.catekv_checked_build():
        pytest.skip("needs the checked build: pytest --checked")
    B, Hkv, G = 1, 2, 4
    lens = [512, 512]
    oc = H.random_cache(B, Hkv, lens, seed=95)
    cache = H.device_cache_from_oracle(ck, oc, max_new=0)      # capacities 512, 512
    n_sel = 64
    rows = np.arange(n_sel, dtype=np.int32) * 7                # rows 0 .. 441 of the segment
    bad = rows.copy()
    bad[10] = 700                                              # row 188 of the NEXT segment: outside [0, 512)
    bad[11] = -3
    idx = torch.from_numpy(np.stack([bad, rows])).cuda()
    sel = torch.tensor([n_sel, n_sel], dtype=torch.int32, device="cuda")
    view = ck.CacheView(cache, [n_sel, n_sel])
    plan = ck.DecodePlan(view, 3)
    ck.catekv_decode_plan(view, plan)
    q = synth.randn_bf16((B, Hkv * G, 128), "cuda", 95, "q")
    out = torch.empty((B, Hkv * G, 128), dtype=torch.float32, device="cuda")
    ck.catekv_checked_status(clear=True)
    ck.catekv_decode_attn_indexed(cache, idx, sel, q, plan, out)
    st = ck.catekv_checked_status(clear=True)
    assert st["flags"] & ck.STATUS_INDEX_RANGE and st["kernel"] == 4 and st["segment"] == 0 and st["index"] in (700, -3)
    # what was read instead: the clamped rows (511 and 0) of segment 0 - the result equals the oracle on that list
    clamped = bad.copy()
    clamped[10], clamped[11] = 511, 0
    soc = orc.HybridCache(B, Hkv, 128)
    kp = synth.bits(cache.k_pool[:512])
    vp = synth.bits(cache.v_pool[:512])
    soc.k_rows = [kp[clamped], oc.k_rows[1][rows]]
    soc.v_rows = [vp[clamped], oc.v_rows[1][rows]]
    ref, _ = orc.decode_attention(soc, synth.bits(q))
    H.check_attention(out, None, None, ref, None, "clamped list")
