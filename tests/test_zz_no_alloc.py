"""catekv_decode_attn_noalloc: the decode call for callers that cannot provide scratch memory.

Some users of the library run where device allocations are off limits: the host application has
claimed the GPU's memory up front and hands out none, or the call sits on a serving path where a
cudaMalloc would stall every stream of the device.  For them the library keeps the split-KV partials
in a fixed 4 MiB array of its own.  This file checks, through the C ABI, that the variant gives the
same outputs as catekv_decode_attn (same tolerance as the other decode tests) on two calls in a row,
that the array's stale contents from the first call do not leak into the second, and that a plan too
large for the array is refused.  It is named to be collected last.
"""
import numpy as np
import pytest
import torch

from workloads import synth
import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ck():
    import paper_2608_30295_b200 as pkg
    assert torch.cuda.is_available()
    return pkg.binding


def _case(ck, lens, B, Hkv, G, seed, num_ctas):
    oc = H.random_cache(B, Hkv, lens, seed=seed)
    cache = H.device_cache_from_oracle(ck, oc, 0)
    plan = ck.DecodePlan(cache, num_ctas)
    ck.catekv_decode_plan(cache, plan)
    q = synth.randn_bf16((B, Hkv * G, 128), "cuda", seed, "q")
    return cache, plan, q


def test_noalloc_matches_decode_attn_twice_in_a_row(ck):
    # first call: many pieces per segment; second call: another cache, fewer and different pieces,
    # so that it would pick up the first call's partials if it read a slot it had not written
    cases = [_case(ck, [3000, 64, 1500, 1, 777, 0, 2049, 300], 2, 4, 4, 51, 96),
             _case(ck, [500, 4096, 17, 900], 1, 4, 7, 52, 40)]
    for cache, plan, q in cases:
        B, Hq, d = q.shape
        want32 = torch.empty((B, Hq, d), dtype=torch.float32, device="cuda")
        want_lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
        want16 = torch.empty((B, Hq, d), dtype=torch.bfloat16, device="cuda")
        ck.catekv_decode_attn(cache, q, plan, want32, want_lse)
        ck.catekv_decode_attn(cache, q, plan, want16)
        plan.ws.fill_(0xFF)  # the variant must not depend on the caller workspace
        got32 = torch.full_like(want32, float("nan"))
        got_lse = torch.full_like(want_lse, float("nan"))
        got16 = torch.full_like(want16, float("nan"))
        ck.catekv_decode_attn_noalloc(cache, q, plan, got32, got_lse)
        ck.catekv_decode_attn_noalloc(cache, q, plan, got16)
        torch.cuda.synchronize()
        w32, g32 = want32.cpu().double().numpy(), got32.cpu().double().numpy()
        assert not np.isnan(g32).any()
        assert H.rel_l2(g32, w32) <= H.REL_L2 and H.max_abs(g32, w32) <= H.MAX_ABS
        w16, g16 = want16.float().cpu().double().numpy(), got16.float().cpu().double().numpy()
        assert H.rel_l2(g16, w16) <= H.REL_L2 and H.max_abs(g16, w16) <= H.MAX_ABS
        wl, gl = want_lse.cpu().numpy(), got_lse.cpu().numpy()
        assert np.array_equal(np.isfinite(wl), np.isfinite(gl))
        assert np.allclose(gl[np.isfinite(wl)], wl[np.isfinite(wl)], atol=1e-3)
        # same kernels, same plan: in fact the results are identical
        assert torch.equal(got32, want32) and torch.equal(got16, want16)


def test_noalloc_refuses_a_plan_beyond_the_fixed_array(ck):
    # (num_ctas + B*Hkv) slots of 4128 bytes must fit 4 MiB: 1016 slots at most
    cache, plan, q = _case(ck, [5000, 5000], 1, 2, 4, 53, 1015)
    out = torch.zeros((1, 8, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_decode_attn_noalloc(cache, q, plan, out)
    assert e.value.code == ck.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.all(out == 0)  # nothing ran
    cache, plan, q = _case(ck, [5000, 5000], 1, 2, 4, 53, 1014)  # 1016 slots: the largest that fits
    want = torch.empty_like(out)
    ck.catekv_decode_attn(cache, q, plan, want)
    ck.catekv_decode_attn_noalloc(cache, q, plan, out)
    torch.cuda.synchronize()
    assert torch.equal(out, want)
