"""GPU parity: catekv_head_cv against the CPU oracle, and the head mask it leads to."""
import numpy as np
import pytest
import torch

from oracle import catekv_oracle as orc
from workloads import synth

pytestmark = pytest.mark.gpu

CV_RTOL = 1e-3  # fp32 scores against the fp64 oracle: entries at the percentile threshold may flip


@pytest.fixture(scope="module")
def ck():
    import paper_2608_30295_b200 as pkg
    assert torch.cuda.is_available()
    return pkg.binding


def _cv_both(ck, q, k, seq_len, L_obs, L_init, L_rec, kq, alpha, causal):
    got = ck.catekv_head_cv(q.cuda(), k.cuda(), seq_len, L_init, L_rec, kq, alpha, causal).cpu().numpy()
    want = orc.head_cv(synth.bits(q), synth.bits(k), seq_len, L_obs, L_init, L_rec, float(np.float32(kq)),
                       float(np.float32(alpha)), causal)
    return got, want


@pytest.mark.parametrize("Hq,Hkv,L_obs,n,L_init,L_rec,kq,alpha,causal", [
    (8, 2, 32, 1000, 16, 32, 0.99, 1.0, False),
    (8, 2, 32, 1000, 16, 4, 0.99, 1.0, True),     # L_rec < L_obs: the causal mask cuts into the matrix
    (28, 4, 64, 2048, 64, 16, 0.996, 1.0, True),  # the paper's window 64, L_init = 2048/32, L_rec = 2048/128
    (14, 2, 64, 1537, 64, 16, 0.984, 0.8, True),
    (4, 4, 16, 300, 0, 0, 0.9, 1.0, True),
    (6, 2, 7, 257, 3, 1, 0.5, 1.0, False),
    (16, 2, 64, 1200, 32, 8, 0.99, 1.0, True),    # G = 8, window 64: the largest supported row count (512)
    (10, 2, 50, 900, 16, 8, 0.99, 1.0, True),     # G = 5: row halves that are multiples of lcm(16, G)
    (2, 2, 64, 700, 8, 64, 0.97, 1.0, False),     # G = 1, window 64, no mask (head-major rows, one unit)
    (8, 2, 64, 1100, 0, 3, 0.99, 1.2, True),      # G = 4, window 64, the mask reaches deep into the matrix
])
def test_head_cv_matches_oracle(ck, Hq, Hkv, L_obs, n, L_init, L_rec, kq, alpha, causal):
    w = synth.scaled(synth.WORKLOADS["cfg4"], Hq=Hq, Hkv=Hkv, L_obs=L_obs, B=1)
    types = (np.arange(Hkv) % 2).astype(np.uint8)
    q, k = synth.calibration_prompt(w, 0, 0, n, types)
    got, want = _cv_both(ck, q, k, [n], L_obs, L_init, L_rec, kq, alpha, causal)
    np.testing.assert_allclose(got, want, rtol=CV_RTOL, atol=1e-6)


def test_head_cv_batch_with_ragged_lengths(ck):
    w = synth.scaled(synth.WORKLOADS["cfg4"], Hq=8, Hkv=2, L_obs=32, B=1)
    qs, ks = [], []
    for pr in range(3):
        q, k = synth.calibration_prompt(w, 0, pr, 1200, np.array([1, 0], dtype=np.uint8))
        qs.append(q), ks.append(k)
    q, k = torch.cat(qs), torch.cat(ks)
    seq = [1200, 900, 1031]
    # the window of a shorter sequence is still q's rows; only the keys beyond seq_len are ignored
    got, want = _cv_both(ck, q, k, seq, 32, 16, 8, 0.99, 1.0, True)
    np.testing.assert_allclose(got, want, rtol=CV_RTOL)


def test_head_mask_reproduces_oracle(ck):
    # calibration prompts with planted head types: device scores -> library vote == oracle scores -> oracle vote
    w = synth.scaled(synth.WORKLOADS["cfg4"], B=1)
    layers, prompts, n = 2, 4, 4096
    rng = np.random.default_rng(40)
    types = np.stack([rng.permutation(np.array([1, 1, 0, 0], dtype=np.uint8)) for _ in range(layers)])
    got = np.zeros((prompts, layers * w.Hkv), dtype=np.float32)
    want = np.zeros((prompts, layers * w.Hkv))
    for pr in range(prompts):
        for l in range(layers):
            q, k = synth.calibration_prompt(w, l, pr, n, types[l])
            g, o = _cv_both(ck, q, k, [n], w.L_obs, 64, 16, 0.99, 1.0, True)
            got[pr, l * w.Hkv:(l + 1) * w.Hkv] = g[0]
            want[pr, l * w.Hkv:(l + 1) * w.Hkv] = o[0]
    np.testing.assert_allclose(got, want, rtol=CV_RTOL)
    mask = ck.catekv_classify_heads(got, 0.5)
    assert np.array_equal(mask, orc.static_head_mask(want, 0.5))
    assert np.array_equal(mask, types.reshape(-1))


@pytest.mark.parametrize("L_rec,kq,alpha", [(64, 0.99, 1.0), (4, 0.9, 1.0), (4, 0.5, 0.8)])
def test_head_cv_when_the_entries_crowd_into_one_bin(ck, L_rec, kq, alpha):
    """Zero queries: every window row attends uniformly, so all entries of the matrix are 1 / (visible keys of the
    row) and share one bin of the percentile kernel's first histogram; a CTA's part of it exceeds its list and the
    general radix path runs.  With L_rec < L_obs the causal mask gives the rows different key counts (a few dozen
    distinct values and zeros), else all entries are equal and the score is 0."""
    Hq, Hkv, L_obs, n, L_init = 8, 2, 64, 2400, 16
    w = synth.scaled(synth.WORKLOADS["cfg4"], Hq=Hq, Hkv=Hkv, L_obs=L_obs, B=1)
    q, k = synth.calibration_prompt(w, 0, 0, n, np.array([1, 0], dtype=np.uint8))
    q = torch.zeros_like(q)
    got, want = _cv_both(ck, q, k, [n], L_obs, L_init, L_rec, kq, alpha, True)
    np.testing.assert_allclose(got, want, rtol=CV_RTOL, atol=1e-6)
    if L_rec >= L_obs:
        assert np.all(got == 0.0)
