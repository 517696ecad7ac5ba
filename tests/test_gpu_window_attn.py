"""GPU parity: the prefill attention rows of the observation window (catekv_window_attn) and the selection that takes
their normaliser instead of its own first pass over K."""
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


def _oracle(qw, k, v, seq_len, G, L_obs, cells):
    """out [B,Hq,L_obs,d], lse, lse_scored [B,Hq,L_obs] (NaN outside `cells`)."""
    B, Hq = qw.shape[:2]
    out = np.full(qw.shape, np.nan)
    lse = np.full((B, Hq, L_obs), np.nan)
    lse_sc = np.full((B, Hq, L_obs), np.nan)
    for (b, h) in cells:
        n = int(seq_len[b])
        o, l = orc.window_attention(qw[b, h * G:(h + 1) * G], k[b, h, :n], v[b, h, :n], L_obs)
        out[b, h * G:(h + 1) * G], lse[b, h * G:(h + 1) * G] = o, l
        if n > L_obs:
            lse_sc[b, h * G:(h + 1) * G] = orc.scored_range_lse(qw[b, h * G:(h + 1) * G], k[b, h, :n], L_obs)
        else:
            lse_sc[b, h * G:(h + 1) * G] = -np.inf
    return out, lse, lse_sc


def _inputs(w):
    """Prefill tensors of the workload; plain random ones where the context is too short to plant heavy keys."""
    if w.n >= w.sink + w.local + 2 * synth.N_HEAVY:
        return synth.prefill_layer(w, 0)
    return {"q_win": synth.randn_bf16((w.B, w.Hq, w.L_obs, w.d), "cpu", w.seed, "qw"),
            "k": synth.randn_bf16((w.B, w.Hkv, w.n, w.d), "cpu", w.seed, "k"),
            "v": synth.randn_bf16((w.B, w.Hkv, w.n, w.d), "cpu", w.seed, "v")}


def _check(ck, w, seq_len, cells=None, where=""):
    p = _inputs(w)
    qw, k, v = p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda()
    out, lse, lse_sc = ck.catekv_window_attn(qw, k, v, seq_len)
    out16, _, _ = ck.catekv_window_attn(qw, k, v, seq_len, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    cells = cells if cells is not None else [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    ref, ref_lse, ref_sc = _oracle(synth.bits(p["q_win"]), synth.bits(p["k"]), synth.bits(p["v"]), seq_len, w.G, w.L_obs, cells)
    d = w.d
    H.check_attention(out.reshape(-1, d), out16.reshape(-1, d), lse.reshape(-1), ref.reshape(-1, d), ref_lse.reshape(-1), where)
    ok = ~np.isnan(ref_sc)
    g, r = lse_sc.cpu().double().numpy()[ok], ref_sc[ok]
    fin = np.isfinite(r)
    assert np.array_equal(np.isfinite(g), fin), where
    assert np.all(np.abs(g[fin] - r[fin]) <= 1e-3), (where, np.abs(g[fin] - r[fin]).max())
    return p, lse_sc


@pytest.mark.parametrize("G,L_obs,n", [(4, 32, 1500), (1, 32, 700), (7, 16, 1111), (8, 16, 513), (2, 64, 3000),
                                       (4, 32, 32), (4, 32, 33), (4, 32, 129)])
def test_window_attention_matches_oracle(ck, G, L_obs, n):
    w = synth.scaled(synth.WORKLOADS["cfg0"], B=2, Hq=2 * G, Hkv=2, n=max(n, L_obs), L_obs=L_obs, local=max(64, L_obs),
                     seed=300 + G)
    seq_len = [w.n, max(L_obs, w.n - 77)]
    _check(ck, w, seq_len, where=f"G={G} L_obs={L_obs} n={n}")


def test_window_attention_more_rows_than_one_tile(ck):
    # 7 heads x 64 window rows = 448 query rows: four 128-row tiles per (sequence, KV head)
    w = synth.scaled(synth.WORKLOADS["cfg4"], B=1, n=2500, seed=310)
    _check(ck, w, [w.n], where="G=7 L_obs=64")


def test_select_from_the_prefill_normaliser_equals_its_own_first_pass(ck):
    """catekv_select_compact with row_lse_scored: same kept lists (band-aware against the oracle), and the scores
    behind them equal those of the two-pass call up to the normaliser's rounding."""
    w = synth.scaled(synth.WORKLOADS["cfg0"], B=2, n=5000, budget=300, seed=320)
    p = synth.prefill_layer(w, 0)
    mask = p["head_mask"]
    qw, k, v = p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda()
    seq_len = [w.n, 3777]
    _, _, lse_sc = ck.catekv_window_attn(qw, k, v, seq_len)
    lens = []
    for b in range(w.B):
        lens += [w.budget if mask[b, h] else seq_len[b] for h in range(w.Hkv)]
    kb, qb = synth.bits(p["k"]), synth.bits(p["q_win"])
    for mode, param in ((orc.POOL_NONE, 0), (orc.POOL_SLIDING, 7), (orc.POOL_CHUNK, 8)):
        got = {}
        for given in (False, True):
            cache = ck.Cache(w.B, w.Hkv, lens, 0, "cuda")
            idx = torch.full((w.B * w.Hkv, w.n), -1, dtype=torch.int32, device="cuda")
            ws = ck.catekv_select_compact(qw, k, v, seq_len, mask, cache, w.budget, 1.0, w.sink, w.local, mode, param,
                                          idx_out=idx, row_lse_scored=lse_sc if given else None)
            if cache.struct.reserved:
                ck.catekv_cache_sync_lengths(cache)
            assert ck.catekv_workspace_status(ws)["flags"] == 0
            got[given] = (cache, idx.cpu().numpy())
        for b in range(w.B):
            n = seq_len[b]
            for h in range(w.Hkv):
                if not mask[b, h]:
                    continue
                s = b * w.Hkv + h
                C = orc.window_scores(qb[b, h * w.G:(h + 1) * w.G], kb[b, h, :n], w.L_obs)
                for given in (False, True):
                    cache, idx = got[given]
                    L = int(cache.seg_len[s])
                    H.check_indices_band(idx[s, :L], C, n, w.sink, w.local, w.budget, mode, param, f"given={given} b{b} h{h}")
                    o = int(cache.seg_off[s])
                    assert np.array_equal(synth.bits(cache.k_pool[o:o + L]), kb[b, h][idx[s, :L]])


def test_window_attention_arguments_are_checked_before_any_launch(ck):
    w = synth.scaled(synth.WORKLOADS["cfg0"], n=256)
    p = synth.prefill_layer(w, 0)
    qw, k, v = p["q_win"].cuda(), p["k"].cuda(), p["v"].cuda()
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_window_attn(qw, k, v, [w.L_obs - 1])   # shorter than the window
    assert e.value.code == ck.ERR_INVALID_ARG
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_window_attn(qw, k, v, [w.n], ws=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.code == ck.ERR_WORKSPACE
