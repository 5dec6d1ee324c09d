"""Pins of the oracle's per-codeword (adversarial-model) error correction."""

import numpy as np
import pytest

from oracle.code import chebyshev_points, powers
from oracle.locate import (CORRECTED, DECODE_FAILURE, NO_ERROR, TOL_FP64, locate_exhaustive,
                           locate_subspace)
from oracle.perpos import correct_positions


def _codewords(P, Q, L, seed, points=None):
    rng = np.random.default_rng(seed)
    b = chebyshev_points(P) if points is None else np.asarray(points, dtype=np.float64)
    return powers(b, Q) @ rng.standard_normal((Q, L)), b


def test_majority_vote_is_the_replication_special_case():
    """Q = 1, P = 3: the code is three copies of one value and one error per position is the
    textbook majority vote."""
    Z = np.array([[5.0, -2.0, 0.5, 7.0],
                  [5.0, -2.0, 9.0, 7.0],
                  [7.0, -2.0, 0.5, 7.0]])
    r = correct_positions(Z, chebyshev_points(3), 1, TOL_FP64)
    assert r.outcome == CORRECTED and r.n_active == 2 and r.n_corrected == 2 and r.n_entries == 2
    assert np.allclose(r.corrected, [[5, -2, 0.5, 7]] * 3, atol=1e-12)
    assert list(r.errors_at) == [1, 0, 1, 0] and list(r.touched) == [False, True, True]


def test_line_through_four_points_by_hand():
    """Q = 2, P = 4, points -1, 0, 1, 2: values of 2x + 1 are (-1, 1, 3, 5); one wrong value is the
    one point off the line through the other three (t = 1)."""
    pts = np.array([-1.0, 0.0, 1.0, 2.0])
    for bad in range(4):
        z = np.array([-1.0, 1.0, 3.0, 5.0])
        z[bad] += 0.75
        r = correct_positions(z[:, None], pts, 2, TOL_FP64)
        assert r.outcome == CORRECTED and r.max_errors == 1
        assert list(np.flatnonzero(r.touched)) == [bad]
        assert np.allclose(r.corrected[:, 0], [-1, 1, 3, 5], atol=1e-12)


@pytest.mark.parametrize("P,Q", [(12, 6), (11, 6), (9, 3)])
def test_corrects_floor_half_parity_errors_per_position(P, Q):
    """Lemma (real-number error correction under the adversarial model): any floor((P-Q)/2) errors
    of arbitrary value in one codeword are corrected; the supports differ from position to position
    and cover more nodes than the node-level decision could give up."""
    t = (P - Q) // 2
    L = 300
    Z0, b = _codewords(P, Q, L, seed=P * 10 + Q)
    rng = np.random.default_rng(1)
    Z = Z0.copy()
    sizes = rng.integers(0, t + 1, size=L)
    for l in range(L):
        nodes = rng.choice(P, size=sizes[l], replace=False)
        Z[nodes, l] += rng.choice([-1.0, 1.0], size=sizes[l]) * rng.uniform(0.5, 20.0, size=sizes[l])
    r = correct_positions(Z, b, Q, TOL_FP64)
    assert r.outcome == CORRECTED and r.n_failed == 0
    assert np.array_equal(r.errors_at, sizes) and r.n_entries == sizes.sum() and r.max_errors == t
    assert np.abs(r.corrected - Z0).max() < 1e-9
    assert r.touched.all()
    # the node-level decision (one support for all positions) has to give up on the same data
    assert locate_subspace(Z, b, Q, TOL_FP64).outcome == DECODE_FAILURE


def test_one_error_too_many_is_reported_not_miscorrected():
    P, Q = 10, 4                                           # t = 3
    Z0, b = _codewords(P, Q, 40, seed=5)
    rng = np.random.default_rng(6)
    Z = Z0.copy()
    Z[[0, 3, 5, 8], 7] += rng.uniform(1.0, 2.0, size=4)    # four errors in position 7
    Z[[1, 2], 20] += 3.0                                   # two in position 20
    r = correct_positions(Z, b, Q, TOL_FP64)
    assert r.outcome == DECODE_FAILURE and r.n_active == 2 and r.n_failed == 1 and r.n_corrected == 1
    assert r.errors_at[7] == -1 and r.errors_at[20] == 2
    assert np.array_equal(r.corrected[:, 7], Z[:, 7])       # untouched
    assert np.abs(r.corrected[:, 20] - Z0[:, 20]).max() < 1e-10


def test_single_codeword_agrees_with_exhaustive_node_search():
    """With one position the two definitions coincide: the sparsest support explaining H z."""
    P, Q = 9, 5
    Z0, b = _codewords(P, Q, 1, seed=4)
    for nodes in [(0, 5), (2, 3), (7, 8), (4,)]:
        Z = Z0.copy()
        Z[list(nodes), 0] += np.linspace(1.0, -2.5, len(nodes))
        ex = locate_exhaustive(Z, b, Q, TOL_FP64)
        r = correct_positions(Z, b, Q, TOL_FP64)
        assert sorted(np.flatnonzero(ex.flagged)) == sorted(np.flatnonzero(r.touched)) == list(nodes)
        assert np.abs(r.corrected - Z0).max() < 1e-10


def test_clean_and_nonfinite_positions():
    P, Q = 8, 4
    Z0, b = _codewords(P, Q, 16, seed=9)
    r = correct_positions(Z0, b, Q, TOL_FP64)
    assert r.outcome == NO_ERROR and r.n_active == 0 and np.array_equal(r.corrected, Z0) and not r.touched.any()
    Z = Z0.copy()
    Z[2, 5] = np.inf
    r = correct_positions(Z, b, Q, TOL_FP64)
    assert r.outcome == DECODE_FAILURE and r.n_failed == 1 and r.errors_at[5] == -1
    assert np.array_equal(np.delete(r.corrected, 5, axis=1), np.delete(Z0, 5, axis=1))
    # FP32-stored outputs stay below the FP32 zero tolerance
    from oracle.locate import TOL_FP32
    assert correct_positions(Z0.astype(np.float32), b, Q, TOL_FP32).outcome == NO_ERROR
