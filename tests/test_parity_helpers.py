"""CPU checks of the comparison rules the GPU parity tests rely on (tests/parity.py): which
differences between two rankings count as near-ties, and that every accepted tie is logged."""
import numpy as np

import parity as P


def test_inverted_pairs_lists_exactly_the_pairs_ordered_differently():
    ref = np.array([0.50, 0.40, 0.30, 0.20])
    same = ref * (1 + 1e-6)
    assert P.inverted_pairs(ref, same) == []
    swapped = np.array([0.50, 0.29, 0.30, 0.20])          # shots 1 and 2 change places
    inv = P.inverted_pairs(ref, swapped)
    assert [(i, j) for i, j, _ in inv] == [(1, 2)]
    assert abs(inv[0][2] - 0.25) < 1e-12                   # |0.40 - 0.30| / 0.40
    # equal scores rank by index on both sides: an exact tie that stays a tie is no inversion
    assert P.inverted_pairs(np.array([1.0, 1.0]), np.array([1.0, 1.0])) == []
    assert [(i, j) for i, j, _ in P.inverted_pairs(np.array([1.0, 1.0]), np.array([0.9, 1.0]))] == [(0, 1)]


def test_near_tie_only_accepts_twice_the_score_tolerance_and_nothing_wider():
    ref = np.array([1.000, 1.003, 0.5])                    # 3e-3 apart: inside 2 x 2e-3
    gpu = np.array([1.002, 1.001, 0.5])
    assert P.near_tie_only(ref, gpu)
    ref = np.array([1.000, 1.010, 0.5])                    # 1e-2 apart: a real difference
    gpu = np.array([1.020, 1.010, 0.5])
    assert not P.near_tie_only(ref, gpu)


def test_accepted_ties_are_logged_with_their_gaps():
    n = len(P.TIE_LOG)
    P.report_tie("unit (b=0, l=1)", 2, 1e-9, 3e-4)
    assert len(P.TIE_LOG) == n + 1
    t = P.TIE_LOG.pop()
    assert t["pairs"] == 2 and t["closest_rel_gap"] == 1e-9 and t["widest_rel_gap"] == 3e-4 and "l=1" in t["where"]
