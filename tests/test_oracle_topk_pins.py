"""Pins for the top-k selection oracle: hand-worked cases, brute force with a comparison
function, and the properties the definition fixes."""
import functools
import itertools

import numpy as np

from oracle.topk import topk_batch, topk_positions


def test_hand_worked_ties_take_the_lowest_positions():
    s = [1.0, 3.0, 3.0, 2.0, 3.0]
    assert topk_positions(s, 5, 1).tolist() == [1]
    assert topk_positions(s, 5, 2).tolist() == [1, 2]
    assert topk_positions(s, 5, 3).tolist() == [1, 2, 4]
    assert topk_positions(s, 5, 4).tolist() == [1, 2, 3, 4]
    assert topk_positions(s, 5, 9).tolist() == [0, 1, 2, 3, 4]
    assert topk_positions(s, 3, 2).tolist() == [1, 2]          # only the first M scores count
    assert topk_positions(s, 0, 2).tolist() == []


def test_nans_of_either_sign_are_equal_and_ordered_by_position():
    neg_nan = np.array([0xFFC00000], dtype=np.uint32).view(np.float32)[0]      # NaN with the sign bit set
    pos_nan = np.float32(np.nan)
    assert np.signbit(neg_nan) and np.isnan(neg_nan) and not np.signbit(pos_nan)
    s = np.array([neg_nan, 1.0, pos_nan, neg_nan, pos_nan], dtype=np.float32)
    # one number, then the NaNs in order of position, whatever their sign bits
    assert topk_positions(s, 5, 1).tolist() == [1]
    assert topk_positions(s, 5, 2).tolist() == [0, 1]
    assert topk_positions(s, 5, 3).tolist() == [0, 1, 2]
    assert topk_positions(s, 5, 4).tolist() == [0, 1, 2, 3]


def test_hand_worked_zero_signs_nan_and_infinities():
    s = np.array([0.0, -0.0, np.nan, -1.0, np.inf, -np.inf], dtype=np.float32)
    assert topk_positions(s, 6, 1).tolist() == [4]
    assert topk_positions(s, 6, 2).tolist() == [0, 4]
    assert topk_positions(s, 6, 3).tolist() == [0, 1, 4]
    assert topk_positions(s, 6, 4).tolist() == [0, 1, 3, 4]
    assert topk_positions(s, 6, 5).tolist() == [0, 1, 3, 4, 5]  # NaN goes last
    assert topk_positions(s, 6, 6).tolist() == [0, 1, 2, 3, 4, 5]


def _ranks_before(a, b):
    """comparison on (score, position): negative when a comes first in the order of the definition"""
    (x, i), (y, j) = a, b
    xn, yn = np.isnan(x), np.isnan(y)
    if xn != yn:
        return 1 if xn else -1
    if not xn:
        if x > y:
            return -1
        if x < y:
            return 1
        sx, sy = np.signbit(x), np.signbit(y)
        if sx != sy:
            return 1 if sx else -1
    return -1 if i < j else (1 if i > j else 0)


def test_brute_force_with_a_comparison_function_on_small_alphabets():
    alphabet = [np.float32(v) for v in (-1.5, -0.0, 0.0, 2.0, np.nan, np.inf)]
    for M in (1, 2, 3, 4):
        for combo in itertools.product(alphabet, repeat=M):
            ordered = sorted(zip(combo, range(M)), key=functools.cmp_to_key(_ranks_before))
            for k in range(1, M + 2):
                want = sorted(i for _, i in ordered[:k])
                assert topk_positions(np.array(combo, dtype=np.float32), M, k).tolist() == want


def test_distinct_scores_agree_with_a_plain_sort_and_separate_the_two_sides():
    rng = np.random.default_rng(7)
    for M, k in ((1, 1), (10, 3), (1000, 64), (5000, 4999)):
        s = rng.permutation(M).astype(np.float32) - M / 3
        got = topk_positions(s, M, k)
        assert set(got.tolist()) == set(np.argsort(s)[M - k:].tolist())
        assert np.all(np.diff(got) > 0)
        rest = np.setdiff1d(np.arange(M), got)
        if len(rest):
            assert s[got].min() > s[rest].max()


def test_quantised_scores_threshold_properties():
    rng = np.random.default_rng(8)
    M, k = 3000, 500
    s = rng.integers(0, 6, M).astype(np.float32)
    got = topk_positions(s, M, k)
    assert len(got) == k and np.all(np.diff(got) > 0)
    thr = s[got].min()
    rest = np.setdiff1d(np.arange(M), got)
    assert s[rest].max() <= thr
    # every score above the threshold is in; the threshold ties kept are the earliest ones
    assert set(np.nonzero(s > thr)[0].tolist()) <= set(got.tolist())
    ties_in = [i for i in got.tolist() if s[i] == thr]
    ties_all = np.nonzero(s == thr)[0].tolist()
    assert ties_in == ties_all[: len(ties_in)]


def test_batch_form_pads_and_clamps():
    s = np.array([[5, 1, 4, 2], [9, 8, 7, 6]], dtype=np.float32)
    idx, ln = topk_batch(s, [4, 2], 3)
    assert ln.tolist() == [3, 2]
    assert idx.tolist() == [[0, 2, 3], [0, 1, -1]]
    idx, ln = topk_batch(s, [0, 99], 2)
    assert ln.tolist() == [0, 2] and idx[1].tolist() == [0, 1]
