"""Pins for the oracle's head identification (Eq. 1-5 and the static vote).  CPU only."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import catekv_oracle as orc
from workloads import synth
from test_oracle_attention import _golden


def test_cv_hand_example(golden_dir):
    g = _golden(golden_dir, "hand_examples.txt")
    A = np.array([[.7, .1, .1, .1], [.6, .2, .1, .1]])
    assert orc.quantile_lower(A, 0.75) == 0.2
    phi = orc.quantile_lower(A, 0.75) * 1.0
    C = (A >= phi).sum(axis=0)
    assert list(C) == [int(x) for x in g["cv_C"]]
    cv = orc.cv_from_matrix(A, 0.75, 1.0)
    assert abs(cv * cv - float(Fraction(g["cv_squared"][0]))) < 1e-14
    assert abs(cv - 1.105542) < 5e-7


def test_quantile_is_numpy_lower():
    rng = np.random.default_rng(20)
    for shape, k in [((7, 13), 0.99), ((64, 50), 0.996), ((3, 3), 0.5), ((1, 1), 0.3), ((10, 10), 0.0),
                     ((10, 10), 1.0), ((64, 200), 0.984)]:
        A = rng.random(shape)
        assert orc.quantile_lower(A, k) == np.quantile(A.reshape(-1), k, method="lower")


def test_cv_closed_forms():
    L_obs, m = 64, 1000
    # all rows identical with c columns above the threshold -> C = L_obs on c columns -> sqrt(m/c - 1)
    for c in (1, 10, 37):
        A = np.full((L_obs, m), 1e-4)
        A[:, :c] = 0.5
        # quantile index N - c*L_obs: the lowest-ranked of the large entries
        k = 1.0 - (c * L_obs - 1) / (L_obs * m - 1) + 1e-12
        cv = orc.cv_from_matrix(A, k, 1.0)
        assert cv == pytest.approx(math.sqrt(m / c - 1), rel=1e-12), (c, k)
    # T ones in distinct columns (each row marks its own columns) -> sqrt(m/T - 1)
    A = np.full((L_obs, m), 1e-4)
    per_row = 5
    for i in range(L_obs):
        A[i, i * per_row:(i + 1) * per_row] = 0.5
    T = L_obs * per_row
    cv = orc.cv_from_matrix(A, 1.0 - (T - 1) / (L_obs * m - 1) + 1e-12, 1.0)
    assert cv == pytest.approx(math.sqrt(m / T - 1), rel=1e-12)
    # the two patterns bracket the score for k = 0.99, L_obs = 64: T = 0.01*N marks
    # spread over distinct columns -> sqrt(1/(0.01*64) - 1) = 0.75; packed into full columns -> sqrt(99) = 9.95
    assert math.sqrt(1 / (0.01 * 64) - 1) == pytest.approx(0.75)
    assert math.sqrt(1 / 0.01 - 1) == pytest.approx(9.9499, rel=1e-4)
    # alpha above one with a flat matrix: nothing passes, mean 0 -> score 0
    assert orc.cv_from_matrix(np.full((4, 9), 0.1), 0.5, 1.5) == 0.0
    # CV is invariant to a common factor on C: doubling the rows doubles every count
    rng = np.random.default_rng(21)
    A = rng.random((8, 300))
    a = orc.cv_from_matrix(A, 0.9, 1.0)
    b = orc.cv_from_matrix(np.concatenate([A, A]), 0.9, 1.0)
    assert b == pytest.approx(a, rel=1e-9)


def test_cv_against_numpy_statistics():
    rng = np.random.default_rng(22)
    A = rng.random((16, 400)) ** 6
    for k, alpha in [(0.99, 1.0), (0.984, 0.8), (0.5, 1.0)]:
        phi = np.quantile(A.reshape(-1), k, method="lower") * alpha
        C = (A >= phi).sum(axis=0)
        want = np.std(C) / np.mean(C)  # numpy's std is the population one
        assert orc.cv_from_matrix(A, k, alpha) == pytest.approx(want, rel=1e-12)


def test_observation_matrix_against_library_softmax():
    rng = np.random.default_rng(23)
    G, L_obs, n, d, L_init, L_rec = 3, 6, 50, 16, 4, 2
    qw = orc.f64_to_bf16(rng.standard_normal((G, L_obs, d)))
    k = orc.f64_to_bf16(rng.standard_normal((n, d)))
    Q = torch.from_numpy(orc.bf16_to_f64(qw))
    K = torch.from_numpy(orc.bf16_to_f64(k))[L_init:n - L_rec]
    S = torch.einsum("gid,jd->gij", Q, K) / math.sqrt(d)
    want = torch.softmax(S, dim=-1).mean(dim=0).numpy()
    A = orc.observation_matrix(qw, k, L_obs, L_init, L_rec, causal=False)
    assert A.shape == (L_obs, n - L_init - L_rec)
    np.testing.assert_allclose(A, want, rtol=1e-12)
    np.testing.assert_allclose(A.sum(axis=1), 1.0, rtol=1e-12)
    # causal: row i sits at position n - L_obs + i and sees keys up to itself
    key = torch.arange(L_init, n - L_rec)[None, :]
    row = (n - L_obs + torch.arange(L_obs))[:, None]
    Sm = S.masked_fill((key > row)[None], float("-inf"))
    want_c = torch.softmax(Sm, dim=-1).mean(dim=0).numpy()
    Ac = orc.observation_matrix(qw, k, L_obs, L_init, L_rec, causal=True)
    np.testing.assert_allclose(Ac, want_c, rtol=1e-12)
    np.testing.assert_allclose(Ac.sum(axis=1), 1.0, rtol=1e-12)
    # L_rec < L_obs here, so the first rows have masked (zero) entries at the end
    assert Ac[0, -1] == 0.0 and Ac[0, n - L_obs - L_init] > 0 and Ac[0, n - L_obs - L_init + 1] == 0.0
    assert np.all(Ac[-1] > 0)
    # with L_rec >= L_obs no key is ahead of any window row: both readings coincide
    A1 = orc.observation_matrix(qw, k, L_obs, L_init, L_obs, causal=True)
    A2 = orc.observation_matrix(qw, k, L_obs, L_init, L_obs, causal=False)
    assert np.array_equal(A1, A2)


def test_cv_separates_planted_head_types():
    w = synth.scaled(synth.WORKLOADS["cfg4"], Hq=8, Hkv=4, L_obs=16, B=1)
    types = np.array([1, 0, 1, 0], dtype=np.uint8)
    q, k = synth.calibration_prompt(w, 0, 0, 2048, types)
    cv = orc.head_cv(synth.bits(q), synth.bits(k), [2048], 16, 64, 16, 0.99, 1.0, True)[0]
    assert cv[0] > 1.5 * cv[1] and cv[2] > 1.5 * cv[3]
    assert np.array_equal(orc.classify_sample(cv, 0.5), types)


def _brute_classify(s, r):
    H = len(s)
    srt = sorted(s)
    gamma = srt[int(math.floor(r * (H - 1)))]
    return [1 if x > gamma else 0 for x in s]


def test_classification_brute_force_and_counts():
    rng = np.random.default_rng(24)
    for H, r in itertools.product((2, 5, 8), (0.0, 0.3, 0.4, 0.5, 1.0)):
        s = rng.random(H)
        got = orc.classify_sample(s, r)
        assert list(got) == _brute_classify(list(s), r)
        # distinct scores: exactly floor(r (H-1)) + 1 adaptive heads
        assert int((got == 0).sum()) == int(math.floor(r * (H - 1))) + 1
    # ties at the threshold are adaptive (Eq. 5: <= Gamma)
    assert list(orc.classify_sample(np.array([1.0, 2.0, 2.0, 3.0]), 0.5)) == [0, 0, 0, 1]
    # a 2-D score matrix (layers x heads) is classified over all heads at once
    S = np.array([[5.0, 1.0], [2.0, 4.0]])
    assert list(orc.classify_sample(S, 0.4)) == [1, 0, 0, 1]


def test_static_mask_vote():
    # 3 samples, 4 heads; per-sample Eq. 5 with r = 0.5 -> 2 adaptive each
    cv = np.array([[9.0, 1.0, 8.0, 2.0],
                   [9.0, 7.0, 1.0, 2.0],
                   [9.0, 1.0, 8.0, 2.0]])
    # consistent votes: head0 3, head1 1, head2 2, head3 0 -> two consistent heads: 0 and 2
    assert list(orc.static_head_mask(cv, 0.5)) == [1, 0, 1, 0]
    # frequency tie broken by mean score, then by index
    cv2 = np.array([[5.0, 4.0, 1.0, 0.0],
                    [4.0, 5.0, 1.0, 0.0]])
    # r = 0.7: floor(.7*3) = 2 -> gamma = third smallest; only the top head is consistent per sample
    # votes: head0 1, head1 1 -> one consistent head in total; means tie (4.5) -> lower index
    assert list(orc.static_head_mask(cv2, 0.7)) == [1, 0, 0, 0]
    m = orc.static_head_mask(np.random.default_rng(25).random((8, 112)), 0.5)
    assert int((m == 0).sum()) == int(math.floor(0.5 * 111)) + 1
