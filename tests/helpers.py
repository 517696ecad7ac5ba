"""Shared helpers of the library tests: loading oracle caches onto the device and error metrics."""
import math

import numpy as np
import torch

from oracle import catekv_oracle as orc
from workloads import synth

# Tolerances (bf16 inputs, fp32 accumulation): relative L2 <= 1e-3 and max-abs <= 1e-2 on attention
# outputs.  The fp32 output is compared with the oracle's fp64 result, the bf16 output with the oracle's
# result rounded to bf16 (rounding alone costs ~1.7e-3 relative L2, so like is compared with like).
REL_L2 = 1e-3
MAX_ABS = 1e-2
TIE_BAND = 1e-4  # relative gap below which the k-th / (k+1)-th pooled scores count as tied


def rel_l2(got, ref):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / (den if den > 0 else 1.0))


def max_abs(got, ref):
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - np.asarray(ref, dtype=np.float64)))) if np.size(ref) else 0.0


def device_cache_from_oracle(ck, ocache, max_new, device="cuda"):
    """Copy an oracle HybridCache into a device Cache (rows written by torch copies)."""
    lens = ocache.lengths()
    cache = ck.Cache(ocache.B, ocache.Hkv, lens, max_new, device)
    for i in range(ocache.B * ocache.Hkv):
        L = int(lens[i])
        if L:
            o = int(cache.seg_off[i])
            cache.k_pool[o:o + L] = synth.from_bits(ocache.k_rows[i], device)
            cache.v_pool[o:o + L] = synth.from_bits(ocache.v_rows[i], device)
    cache.set_lengths(lens)
    return cache


def random_cache(B, Hkv, lens, seed, d=128):
    """An oracle cache with random rows of the given lengths [B*Hkv]."""
    oc = orc.HybridCache(B, Hkv, d)
    for i, L in enumerate(lens):
        oc.k_rows.append(synth.bits(synth.randn_bf16((int(L), d), "cpu", seed, "k", i)))
        oc.v_rows.append(synth.bits(synth.randn_bf16((int(L), d), "cpu", seed, "v", i)))
    return oc


def _bf16_ordinal(bits):
    """bf16 bit patterns -> integers that are consecutive for adjacent values (+0 and -0 both map to 0)."""
    b = np.asarray(bits).astype(np.int64)
    mag = b & 0x7FFF
    return np.where(b & 0x8000, -mag, mag)


def bf16_tie_flips(got_bits, ref_bits, x_f32, ref_f64):
    """Elements whose bf16 value differs from the rounded oracle value for the one excusable reason: the fp32 result
    x_f32 and the oracle value sit on opposite sides of the midpoint of two adjacent bf16 numbers.

    True where (i) got and ref are adjacent bf16 values and (ii) x lies within TIE_DIST of their midpoint, with
    TIE_DIST = max |x_f32 - ref_f64| over the tensor (the measured fp32 error) + 4 fp32 ulps of x."""
    return bf16_tie_analysis(got_bits, ref_bits, x_f32, ref_f64)[0]


def bf16_tie_analysis(got_bits, ref_bits, x_f32, ref_f64):
    """-> (mask of excused elements, number of such elements to expect).  An fp32 value falls within TIE_DIST of a
    rounding midpoint with probability 2 TIE_DIST / ulp (ulp: the bf16 spacing at that magnitude) when it is spread
    evenly between two bf16 neighbours; the sum of these probabilities is the expected count."""
    differ = np.asarray(got_bits) != np.asarray(ref_bits)
    adjacent = np.abs(_bf16_ordinal(got_bits) - _bf16_ordinal(ref_bits)) == 1
    mid = 0.5 * (orc.bf16_to_f64(got_bits) + orc.bf16_to_f64(ref_bits))
    x = np.asarray(x_f32, dtype=np.float64)
    err = float(np.max(np.abs(x - ref_f64))) if x.size else 0.0
    tie_dist = err + 4.0 * np.spacing(np.abs(x).astype(np.float32)).astype(np.float64)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(np.asarray(ref_f64, dtype=np.float64)), 2.0 ** -126))) - 7)
    expected = float(np.minimum(1.0, 2.0 * tie_dist / ulp).sum())
    return differ & adjacent & (np.abs(x - mid) <= tie_dist), expected


def check_attention(out_f32, out_bf16, lse, ref, ref_lse, where=""):
    """ref: oracle fp64 [.., d]; NaN rows of ref are skipped."""
    ok = ~np.isnan(ref).any(axis=-1)
    r = ref[ok]
    if out_f32 is not None:
        g = out_f32.detach().cpu().double().numpy()[ok]
        assert rel_l2(g, r) <= REL_L2, (where, "fp32 rel-L2", rel_l2(g, r))
        assert max_abs(g, r) <= MAX_ABS, (where, "fp32 max-abs", max_abs(g, r))
    if out_bf16 is not None:
        # The bf16 output is the same arithmetic rounded once at the end: bit-identical to the fp32 output of the
        # same call sequence rounded to nearest-even (which carries the parity claim against the fp64 oracle above).
        assert out_f32 is not None, "a bf16 output is checked together with the fp32 output of the same call"
        assert np.array_equal(synth.bits(out_bf16), synth.bits(out_f32.to(out_bf16.dtype))), (where, "bf16 != rne(fp32)")
        # Against the oracle rounded to bf16 (like with like).  Where the oracle's value and the fp32 result lie on
        # opposite sides of a rounding tie they round to the two neighbours: one bf16 ulp apart (2^-6 for |x| in
        # [2, 4), above the 1e-2 absolute bound).  Such an element is excused only when the cause shows: the two
        # values are adjacent bf16 numbers and the fp32 result lies within TIE_DIST of their midpoint, TIE_DIST =
        # the largest fp32-against-oracle error measured on this tensor + 4 fp32 ulps, and there may be no more of
        # them than that distance explains.  Every other element keeps rel-L2 <= 1e-3 and max-abs <= 1e-2.
        gbits = synth.bits(out_bf16)[ok]
        rbits = orc.f64_to_bf16(r)
        g, rb = orc.bf16_to_f64(gbits), orc.bf16_to_f64(rbits)
        x = out_f32.detach().cpu().double().numpy()[ok]
        tie, expected = bf16_tie_analysis(gbits, rbits, x, r)
        n_ties = int(tie.sum())
        # no more such elements than chance explains: three times the expected count (+ 4 for small tensors)
        assert n_ties <= 4 + 3.0 * expected, (where, "too many rounding-tie flips to be chance", n_ties, expected)
        g_chk = np.where(tie, rb, g)
        assert rel_l2(g_chk, rb) <= REL_L2, (where, "bf16 rel-L2", rel_l2(g_chk, rb), n_ties)
        assert max_abs(g_chk, rb) <= MAX_ABS, (where, "bf16 max-abs", max_abs(g_chk, rb), n_ties)
    if lse is not None:
        gl = lse.detach().cpu().double().numpy()[ok]
        rl = ref_lse[ok]
        fin = np.isfinite(rl)
        assert np.array_equal(np.isfinite(gl), fin), where
        assert np.all(np.abs(gl[fin] - rl[fin]) <= 1e-3), (where, "lse", np.abs(gl[fin] - rl[fin]).max())


def check_indices_band(got_idx, C, n, S, Lc, T, mode, param, where=""):
    """Band-aware comparison of a kept list with the oracle's selection.

    The oracle's pooled scores P (fp64) define the k-th largest value P_k.  The list must be strictly
    ascending, hold the sink and local tokens, have the oracle's length, contain every candidate with
    P > P_k (1 + band) and nothing with P < P_k (1 - band).  Returns True when the oracle's gap around
    the threshold is wide enough that the comparison was bit-exact.
    """
    want = orc.select_indices(C, n, S, Lc, T, mode, param)
    got = np.asarray(got_idx, dtype=np.int64)
    assert got.shape == want.shape, (where, got.shape, want.shape)
    assert np.all(np.diff(got) > 0), where
    if np.array_equal(got, want):
        return True
    assert T < n and S + Lc < n, where
    cand_end = n - Lc
    P = orc.pool_scores(C, S, cand_end, mode, param)
    cs = param if mode == orc.POOL_CHUNK else 1
    k_sel = max(0, T - S - Lc) // cs
    order = np.sort(P)[::-1]
    Pk = order[k_sel - 1]
    assert list(got[:S]) == list(range(S)) and list(got[-Lc:]) == list(range(n - Lc, n)), where
    mid = got[S:len(got) - Lc]
    units = np.unique((mid - S) // cs)
    must = np.nonzero(P > Pk * (1 + TIE_BAND))[0]
    may = np.nonzero(P >= Pk * (1 - TIE_BAND))[0]
    assert set(must.tolist()) <= set(units.tolist()), (where, "missing clear winners")
    assert set(units.tolist()) <= set(may.tolist()), (where, "took a clear loser")
    assert len(units) == k_sel, where
    return False


def check_retrieval_band(got, scores, n, S, Lc, budget, cs, where=""):
    """Band-aware comparison of the rows a retrieval head attends to with the oracle's (fp32 bounds on the device
    against fp64 bounds): same length, ascending, every chunk whose bound is clearly above the k-th largest taken,
    none clearly below it.  Returns True when the lists were identical."""
    want = orc.retrieve_indices(scores, n, S, Lc, budget, cs)
    got = np.asarray(got, dtype=np.int64)
    assert got.shape == want.shape, (where, got.shape, want.shape)
    assert np.all(np.diff(got) > 0), where
    if np.array_equal(got, want):
        return True
    S2 = (S + cs - 1) // cs * cs
    cand_end = (n - Lc) // cs * cs
    P = scores[S2 // cs: cand_end // cs]
    k_sel = (budget - S2 - (n - cand_end)) // cs
    Pk = np.sort(P)[::-1][k_sel - 1]
    tol = TIE_BAND * max(1.0, abs(Pk))
    assert np.array_equal(got[:S2], np.arange(S2)) and np.array_equal(got[len(got) - (n - cand_end):],
                                                                      np.arange(cand_end, n)), where
    mid = got[S2:len(got) - (n - cand_end)]
    assert np.all((mid - S2) % cs == np.tile(np.arange(cs), len(mid) // cs)), (where, "not whole chunks")
    units = np.unique((mid - S2) // cs)
    assert len(units) == k_sel, where
    assert set(np.nonzero(P > Pk + tol)[0].tolist()) <= set(units.tolist()), (where, "missing clear winners")
    assert set(units.tolist()) <= set(np.nonzero(P >= Pk - tol)[0].tolist()), (where, "took a clear loser")
    return False
