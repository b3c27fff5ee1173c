"""The comparison rule the GPU parity tests apply (tests/helpers.match_results), exercised on hand-made lists.

A rule that is too lenient would let wrong results pass every parity test, so its own behaviour is pinned here:
ids may differ from the oracle's only inside distance ties, an id the oracle does not list must be scored by the
oracle itself, and nothing may be returned twice.
"""

import numpy as np

from tests.helpers import match_results


def _o():
    return np.array([5, 9, 2, 7], np.int64), np.array([1.0, 2.0, 3.0, 4.0], np.float32)


def test_identical_lists_match():
    i, d = _o()
    assert not match_results(i, d, i, d)


def test_distance_off_by_more_than_tolerance_is_reported():
    i, d = _o()
    d2 = d.copy()
    d2[2] *= 1.001
    assert match_results(i, d2, i, d, rel=1e-4)
    d2[2] = d[2] * (1 + 5e-5)
    assert not match_results(i, d2, i, d, rel=1e-4)


def test_ids_may_swap_only_inside_a_tie():
    i = np.array([5, 9, 2, 7], np.int64)
    d = np.array([1.0, 2.0, 2.0, 4.0], np.float32)
    assert not match_results(np.array([5, 2, 9, 7]), d, i, d)
    d_apart = np.array([1.0, 2.0, 3.0, 4.0], np.float32)
    assert match_results(np.array([5, 2, 9, 7]), d_apart, i, d_apart)


def test_id_missing_from_the_oracle_list_needs_the_oracle_score():
    i, d = _o()
    mine = np.array([5, 9, 2, 11], np.int64)           # 11 replaces the last entry
    assert match_results(mine, d, i, d)                 # nobody vouches for id 11
    assert not match_results(mine, d, i, d, rescore=lambda ident: 4.0)          # the oracle scores it at the tie
    assert match_results(mine, d, i, d, rescore=lambda ident: 4.5)              # the oracle scores it worse
    assert match_results(mine, d, i, d, rescore=lambda ident: 3.0)              # or better: then it belonged earlier

    def unknown(ident):
        raise KeyError(ident)
    assert match_results(mine, d, i, d, rescore=unknown)                        # an id the index does not hold


def test_an_id_returned_twice_is_reported():
    i, d = _o()
    d_tie = np.array([1.0, 2.0, 2.0, 4.0], np.float32)
    assert match_results(np.array([5, 9, 9, 7]), d_tie, np.array([5, 9, 2, 7]), d_tie, rescore=lambda ident: 2.0)


def test_padding_must_agree():
    i = np.array([5, -1], np.int64)
    d = np.array([1.0, np.inf], np.float32)
    assert not match_results(i, d, i, d)
    assert match_results(np.array([5, 3]), d, i, d)
