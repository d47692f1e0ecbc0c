"""Offline layer-mapping utilities (Sec. 3.3 and App. B, Alg. 3) against brute force and library
routines.  CPU only."""
import itertools

import numpy as np
import pytest
from scipy.stats import entropy

from paper_2510_27641_b200.layer_mapping import kl_similarity, monotonic_dtw


def _brute_force(S):
    m, n = S.shape
    best, best_f = -np.inf, None
    for f in itertools.combinations_with_replacement(range(m), n):     # all non-decreasing maps
        t = sum(S[f[j], j] for j in range(n))
        if t > best:
            best, best_f = t, f
    return best, best_f


@pytest.mark.parametrize("seed", range(12))
def test_monotonic_dtw_equals_exhaustive_search(seed):
    rng = np.random.default_rng(seed)
    m, n = int(rng.integers(1, 6)), int(rng.integers(1, 7))
    S = -rng.random((m, n)) * 5
    f, total = monotonic_dtw(S)
    want, _ = _brute_force(S)
    assert np.all(np.diff(f) >= 0) and f.min() >= 0 and f.max() < m
    assert total == pytest.approx(want, abs=1e-12)
    assert total == pytest.approx(sum(S[f[j], j] for j in range(n)), abs=1e-12)


def test_monotonic_dtw_structure():
    # when the column-wise argmax is already monotone it is the answer
    S = np.full((4, 6), -9.0)
    for j, i in enumerate([0, 0, 1, 3, 3, 3]):                 # draft layer 2 skipped, 0 and 3 repeated
        S[i, j] = -0.5
    f, total = monotonic_dtw(S)
    assert f.tolist() == [0, 0, 1, 3, 3, 3] and total == pytest.approx(-3.0)
    # a decreasing preference cannot be followed: one of the two layers must give way
    S = np.array([[-5.0, -1.0], [-1.0, -5.0]])
    f, total = monotonic_dtw(S)
    assert total == pytest.approx(-6.0) and np.all(np.diff(f) >= 0)
    # equal depths with a dominant diagonal give the identity
    S = -np.ones((5, 5)) + np.eye(5)
    assert monotonic_dtw(S)[0].tolist() == [0, 1, 2, 3, 4]
    # one draft layer serves every verifier layer; no verifier layers: empty map
    assert monotonic_dtw(np.array([[-1.0, -2.0, -3.0]]))[0].tolist() == [0, 0, 0]
    assert monotonic_dtw(np.zeros((3, 0)))[0].shape == (0,)
    # -inf entries are avoided when a finite monotone map exists
    S = np.array([[-1.0, -np.inf], [-np.inf, -2.0]])
    f, total = monotonic_dtw(S)
    assert f.tolist() == [0, 1] and total == -3.0
    with pytest.raises(ValueError):
        monotonic_dtw(np.array([[np.nan]]))


def test_kl_similarity_equals_library_relative_entropy():
    rng = np.random.default_rng(3)
    av = rng.random((4, 50)); av /= av.sum(1, keepdims=True)
    ad = rng.random((3, 50)); ad /= ad.sum(1, keepdims=True)
    S = kl_similarity(av, ad)
    for i in range(3):
        for j in range(4):
            assert S[i, j] == pytest.approx(-entropy(av[j], ad[i]), rel=1e-12)
    assert np.all(S <= 1e-15)                                   # Gibbs: the divergence is >= 0
    assert np.allclose(np.diag(kl_similarity(av, av)), 0.0)     # and 0 against itself
    # zero verifier mass contributes nothing; verifier mass where the draft has none is -inf
    a = np.array([[0.5, 0.5, 0.0]]); b = np.array([[0.25, 0.25, 0.5], [1.0, 0.0, 0.0]])
    S = kl_similarity(a, b)
    assert S[0, 0] == pytest.approx(-np.log(2.0)) and S[1, 0] == -np.inf


def test_end_to_end_layer_map_feeds_select_args():
    # a verifier twice as deep as the draft whose layer 2j and 2j+1 resemble draft layer j
    rng = np.random.default_rng(5)
    ad = rng.random((4, 64)) ** 3; ad /= ad.sum(1, keepdims=True)
    av = np.repeat(ad, 2, axis=0) * (1 + 0.05 * rng.random((8, 64))); av /= av.sum(1, keepdims=True)
    f, _ = monotonic_dtw(kl_similarity(av, ad))
    assert f.tolist() == [0, 0, 1, 1, 2, 2, 3, 3] and f.dtype == np.int32
