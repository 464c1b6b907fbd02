"""The acceptance rules of the parity harness itself, on the CPU: which differences from the oracle a GPU result
may show (boundary ties of a selection, a class decided by a distance gap below resolution) and which it may not."""
import numpy as np
import pytest

from oracle import taskkv_oracle as O


def _P():
    from tests import parity
    return parity


def test_selection_may_differ_only_at_boundary_ties():
    P = _P()
    score = np.array([5.0, 4.0, 3.0, 3.0 * (1 - 2e-6), 1.0, 0.5])
    want = O.top_indices(score, 3)                      # {0, 1, 2}
    assert P.check_selection(np.array([0, 1, 2]), want, score, "same") == 0
    assert P.check_selection(np.array([0, 1, 3]), want, score, "tie") == 1          # 2 <-> 3: gap 2e-6 relative
    with pytest.raises(AssertionError):
        P.check_selection(np.array([0, 1, 4]), want, score, "not a tie")            # 4 is far below the boundary
    with pytest.raises(AssertionError):
        P.check_selection(np.array([0, 1]), want, score, "short")
    with pytest.raises(AssertionError):
        P.check_selection(np.array([0, 1, 1]), want, score, "duplicate")


def test_class_difference_needs_the_deciding_gap_to_be_small():
    P = _P()
    tol = P.CLASS_TIE_REL
    # far -> near: heads 0, 1 | 2 ... ; f = 2, promoted = nearest of the rest
    dist = np.array([9.0, 8.0, 5.0, 4.0, 4.0 * (1 + 1e-6), 2.0, 1.0])
    want = O.semantic_separator(dist, 2, True)
    assert want.tolist() == [1, 1, 0, 0, 0, 0, 2]
    assert P.classes_valid_up_to(dist, want, 2, True, tol)
    # two distances elsewhere in the ranking are within 1e-6 of each other (heads 3 and 4): that does not excuse a
    # swap at the f-th / (f+1)-th rank, whose gap is wide
    swapped = np.array([1, 0, 1, 0, 0, 0, 2], dtype=np.uint8)
    assert not P.classes_valid_up_to(dist, swapped, 2, True, tol)
    # nor a wrong promoted head
    wrong_centre = np.array([1, 1, 0, 0, 0, 2, 0], dtype=np.uint8)
    assert not P.classes_valid_up_to(dist, wrong_centre, 2, True, tol)
    # a swap exactly at the deciding gap, when that gap is below resolution, is a valid answer
    close = np.array([9.0, 8.0, 8.0 * (1 - 1e-6), 4.0, 3.0, 2.0, 1.0])
    assert O.semantic_separator(close, 2, True).tolist() == [1, 1, 0, 0, 0, 0, 2]
    assert P.classes_valid_up_to(close, np.array([1, 0, 1, 0, 0, 0, 2], dtype=np.uint8), 2, True, tol)
    assert not P.classes_valid_up_to(close, np.array([0, 1, 1, 0, 0, 0, 2], dtype=np.uint8), 2, True, tol)
    # the nearest two of the rest within resolution: either may be promoted, nothing else
    near = np.array([9.0, 8.0, 5.0, 4.0, 3.0, 1.0 * (1 + 1e-6), 1.0])
    assert P.classes_valid_up_to(near, np.array([1, 1, 0, 0, 0, 2, 0], dtype=np.uint8), 2, True, tol)
    assert not P.classes_valid_up_to(near, np.array([1, 1, 0, 0, 2, 0, 0], dtype=np.uint8), 2, True, tol)
    # wrong counts are never valid
    assert not P.classes_valid_up_to(dist, np.array([1, 1, 1, 0, 0, 0, 2], dtype=np.uint8), 2, True, tol)
    assert not P.classes_valid_up_to(dist, np.array([1, 1, 0, 0, 0, 0, 0], dtype=np.uint8), 2, True, tol)
    assert not P.classes_valid_up_to(dist, want, 2, False, tol)                     # no promotion asked for
    assert P.classes_valid_up_to(dist, np.array([1, 1, 0, 0, 0, 0, 0], dtype=np.uint8), 2, False, tol)
    # every head heterogeneous: no head is left to promote
    assert P.classes_valid_up_to(dist, np.ones(7, dtype=np.uint8), 7, True, tol)


def test_tie_bound_is_one_per_ten_thousand_selections():
    P = _P()
    rep = P.Report(selected=704512, topt_ties=40, mid_ties=30)
    rep.check_bounds("ok")                                                           # 70 <= 1 + 70
    rep.mid_ties = 32
    with pytest.raises(AssertionError):
        rep.check_bounds("too many")
    rep = P.Report(selected=500)
    rep.class_near_ties, rep.class_diff = 1, {(0, 3): [1, 2]}
    with pytest.raises(AssertionError):
        rep.check_bounds("unnamed class near-tie")
    rep.check_bounds("named", expect_class_ties=[(0, 3)])
