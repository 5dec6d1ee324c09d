"""Pins of the oracle's error locator: exhaustive search, Theorem 3, special cases."""

import itertools
import os

import numpy as np
import pytest

from oracle import inject as inj
from oracle import product as op
from oracle.code import GPCode, FWD, chebyshev_points, parity_check, powers
from oracle.locate import (CORRECTED, DECODE_FAILURE, NO_ERROR, TOL_FP32, TOL_FP64,
                           locate_exhaustive, locate_subspace)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _codewords(P, Q, L, seed):
    """Clean outputs Z = G^T q for random coefficient vectors (one codeword per column)."""
    rng = np.random.default_rng(seed)
    b = chebyshev_points(P)
    return powers(b, Q) @ rng.standard_normal((Q, L)), b


def _corrupt(Z, nodes, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    Z = Z.copy()
    for p in nodes:
        Z[p] += scale * rng.standard_normal(Z.shape[1])       # Error Model 2: whole output, Gaussian
    return Z


def test_splitmix64_reference_outputs():
    want = [int(l.strip(), 16) for l in open(os.path.join(GOLDEN, "splitmix64_seed0.txt"))
            if l.strip() and not l.startswith("#")]
    got = [int(inj.draw(0, c)) for c in range(4)]
    assert got == want


@pytest.mark.parametrize("P,Q", [(7, 4), (8, 5), (9, 5)])
def test_subspace_equals_exhaustive_on_every_pattern(P, Q):
    """All error supports of size 0..P-Q: both forms agree; <= P-Q-1 corrected exactly,
    more declared a decoding failure (Theorem 3, claims 2 and 3)."""
    Z0, b = _codewords(P, Q, 24, seed=P * 100 + Q)
    seed = 0
    for size in range(0, P - Q + 1):
        for nodes in itertools.combinations(range(P), size):
            seed += 1
            Z = _corrupt(Z0, nodes, seed)
            ex = locate_exhaustive(Z, b, Q, TOL_FP64)
            sb = locate_subspace(Z, b, Q, TOL_FP64)
            assert ex.outcome == sb.outcome
            assert np.array_equal(ex.flagged, sb.flagged)
            if size == 0:
                assert ex.outcome == NO_ERROR
            elif size <= P - Q - 1:
                assert ex.outcome == CORRECTED and sorted(np.flatnonzero(ex.flagged)) == list(nodes)
            else:
                assert ex.outcome == DECODE_FAILURE


def test_detection_for_any_number_of_errors():
    """Theorem 3, claim 1: errors are detected whatever their number."""
    P, Q = 10, 6
    Z0, b = _codewords(P, Q, 16, seed=3)
    for size in range(1, P + 1):
        Z = _corrupt(Z0, range(size), seed=size)
        assert locate_subspace(Z, b, Q, TOL_FP64).outcome != NO_ERROR
        assert locate_exhaustive(Z, b, Q, TOL_FP64).outcome != NO_ERROR


def test_adversarial_bound_single_codeword():
    """One codeword (L = 1): floor((P-Q)/2) errors of arbitrary value are located (adversarial-model
    lemma).  The error matrix then has rank 1 < number of errors, so the subspace form finds no
    column of H in the syndrome's range and must get there through its superset search."""
    P, Q = 9, 5
    Z0, b = _codewords(P, Q, 1, seed=4)
    for nodes in [(0, 5), (2, 3), (7, 8)]:
        Z = Z0.copy()
        Z[list(nodes), 0] += np.array([1.0, -2.5])
        ex = locate_exhaustive(Z, b, Q, TOL_FP64)
        assert ex.outcome == CORRECTED and sorted(np.flatnonzero(ex.flagged)) == list(nodes)
        sb = locate_subspace(Z, b, Q, TOL_FP64)
        assert sb.outcome == CORRECTED and np.array_equal(sb.flagged, ex.flagged) and sb.rank == 1
    # a single error in a single codeword is fine for both
    Z = Z0.copy()
    Z[4, 0] += 0.75
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP64)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [4]


@pytest.mark.parametrize("P,Q,L", [(7, 4, 1), (8, 4, 1), (9, 5, 2), (8, 4, 2)])
def test_rank_deficient_patterns_subspace_equals_exhaustive(P, Q, L):
    """Few codewords (L = 1, 2) and every support of size 0..P-Q: the error matrix has rank
    min(size, L), below the number of erroneous nodes for most patterns.  Theorem 3 (claims 2, 3)
    holds per codeword, so up to P-Q-1 errors are still corrected, more are a declared failure,
    and the subspace form (through its superset search) takes the exhaustive form's decision."""
    Z0, b = _codewords(P, Q, L, seed=7 * P + Q + L)
    rng = np.random.default_rng(P * 1000 + Q * 10 + L)
    for size in range(0, P - Q + 1):
        for nodes in itertools.combinations(range(P), size):
            Z = Z0.copy()
            Z[list(nodes), :] += rng.uniform(0.5, 2.0, (size, L)) * rng.choice([-1.0, 1.0], (size, L))
            ex = locate_exhaustive(Z, b, Q, TOL_FP64)
            sb = locate_subspace(Z, b, Q, TOL_FP64)
            assert ex.outcome == sb.outcome, (nodes, ex.outcome, sb.outcome)
            assert np.array_equal(ex.flagged, sb.flagged), nodes
            if size == 0:
                assert ex.outcome == NO_ERROR
            elif size <= P - Q - 1:
                assert ex.outcome == CORRECTED and sorted(np.flatnonzero(ex.flagged)) == list(nodes)
            else:
                assert ex.outcome == DECODE_FAILURE


def test_partly_rank_deficient_pattern_keeps_the_nodes_already_inside():
    """Three erroneous nodes, two of which err in one codeword only (the same one): rank 2 < 3.  The
    third node's column of H lies in the syndromes' range and is kept; the search adds the others."""
    P, Q, L = 12, 6, 40
    Z0, b = _codewords(P, Q, L, seed=21)
    Z = _corrupt(Z0, (4,), seed=22)
    Z[[1, 9], 17] += np.array([3.0, -1.25])
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP64)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [1, 4, 9]
    assert locate_subspace(Z, b, Q, TOL_FP64).rank == 2


def test_fallback_search_is_bounded():
    """The superset search gives up (declared failure) once the supports to try exceed the bound:
    P = 40, one codeword with 6 errors would need C(40,1) + ... + C(40,6) supports."""
    from oracle.locate import MAX_FALLBACK_SUPPORTS
    P, Q = 40, 20
    Z0, b = _codewords(P, Q, 1, seed=23)
    Z = Z0.copy()
    Z[[0, 1], 0] += np.array([1.0, 2.0])
    assert 40 + 780 <= MAX_FALLBACK_SUPPORTS < 40 + 780 + 9880
    r = locate_subspace(Z, b, Q, TOL_FP64)
    assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [0, 1]
    Z[[5, 6, 7, 8], 0] += np.array([1.0, -1.0, 2.0, 0.5])
    assert locate_subspace(Z, b, Q, TOL_FP64).outcome == DECODE_FAILURE


def test_values_whose_square_overflows_are_located():
    """A finite value above about 1e154 has an infinite square; the zero test ||Hz|| <= tau ||z||
    would compare inf with inf and pass.  Such a value (for instance an FP64 exponent-bit flip:
    x * 2^1000) is handled like a non-finite one: its node is flagged up front."""
    P, Q = 10, 6
    Z0, b = _codewords(P, Q, 20, seed=24)
    Z = Z0.copy()
    Z[3, 7] *= 2.0 ** 1000
    assert np.isfinite(Z).all()
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP64)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [3] and r.forced[3]
    Z[5, 2] = -2.0 ** 499.5                                   # still squares inside the FP64 range
    r = locate_subspace(Z, b, Q, TOL_FP64)
    assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [3, 5] and not r.forced[5]
    # the flip itself, through the injector's bit arithmetic: bit 62 of a value below 1
    w = np.array([[0.75]])
    w.view(np.uint64)[0, 0] ^= np.uint64(1 << 62)
    assert np.isfinite(w[0, 0]) and abs(w[0, 0]) > 2.0 ** 900


def test_bitflip_changes_exactly_one_bit_of_one_entry_per_hit_node():
    rng = np.random.default_rng(25)
    for dtype, itype, nbits in ((np.float32, np.uint32, 32), (np.float64, np.uint64, 64)):
        Z0 = rng.standard_normal((9, 6, 5)).astype(dtype)
        for seed in range(30):
            for count in (1, 2, 4, 9, 12):
                Z = Z0.copy()
                hit = inj.inject_bitflip(Z, seed, count, scale=1.0)
                assert hit.sum() == min(count, 9)
                diff = (Z.view(itype) ^ Z0.view(itype)).reshape(9, -1)
                for p in range(9):
                    changed = np.flatnonzero(diff[p])
                    if not hit[p]:
                        assert changed.size == 0
                        continue
                    assert changed.size == 1                                   # one entry
                    assert bin(int(diff[p, changed[0]])).count("1") == 1       # one bit
                    new, old = Z.reshape(9, -1)[p, changed[0]], Z0.reshape(9, -1)[p, changed[0]]
                    assert (not np.isfinite(new)) or abs(float(new) - float(old)) >= 2.0 ** -6


def test_replication_special_case():
    """Q = 1 is replication: with two values still agreeing the P-2 others are corrected;
    with no two agreeing a failure is declared (Section V-A)."""
    P, Q = 5, 1
    rng = np.random.default_rng(5)
    b = chebyshev_points(P)
    Z0 = np.repeat(rng.standard_normal((1, 12)), P, axis=0)
    Z = _corrupt(Z0, (0, 2, 4), seed=6)
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP64)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [0, 2, 4]
    Z = _corrupt(Z0, (0, 1, 2, 4), seed=7)
    for fn in (locate_exhaustive, locate_subspace):
        assert fn(Z, b, Q, TOL_FP64).outcome == DECODE_FAILURE


def test_nonfinite_and_erased_nodes_are_flagged_and_counted():
    P, Q = 10, 6
    Z0, b = _codewords(P, Q, 20, seed=8)
    Z = Z0.copy()
    Z[3, 7] = np.inf
    Z[6, 2] = np.nan
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP64)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [3, 6]
    erased = np.zeros(P, dtype=bool)
    erased[[1, 8]] = True
    Z = _corrupt(Z0, (5,), seed=9)
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP64, erased=erased)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [1, 5, 8]
    erased[[0, 2]] = True                                   # 4 erasures + 1 error > P-Q-1 = 3
    for fn in (locate_exhaustive, locate_subspace):
        assert fn(Z, b, Q, TOL_FP64, erased=erased).outcome == DECODE_FAILURE


def test_fp32_outputs_clean_floor_and_bitflips():
    """Outputs rounded to FP32 stay below the FP32 zero tolerance; two injected bit flips are found."""
    P, Q, L = 13, 9, 1024
    Z0, b = _codewords(P, Q, L, seed=10)
    Z32 = Z0.astype(np.float32)
    assert locate_subspace(Z32, b, Q, TOL_FP32).outcome == NO_ERROR
    for seed in range(20):
        Z = Z32.copy()
        hit = inj.inject_bitflip(Z, seed, 2, scale=float(np.sqrt(np.mean(Z0 ** 2))))
        assert hit.sum() == 2
        changed = np.flatnonzero((Z.view(np.uint32) != Z32.view(np.uint32)).any(axis=1))
        assert list(changed) == list(np.flatnonzero(hit))
        r = locate_subspace(Z, b, Q, TOL_FP32)
        e = locate_exhaustive(Z, b, Q, TOL_FP32)
        assert r.outcome == e.outcome == CORRECTED and np.array_equal(r.flagged, e.flagged)
        assert np.array_equal(r.flagged, hit)
    # both flips in the same codeword (rank 1, two erroneous nodes): floor((13-9)/2) = 2 errors in
    # one codeword are correctable (adversarial-model lemma), through the superset search
    Z = Z32.copy()
    Z.view(np.uint32)[2, 100] ^= np.uint32(1 << 27)
    Z.view(np.uint32)[11, 100] ^= np.uint32(1 << 22)
    for fn in (locate_exhaustive, locate_subspace):
        r = fn(Z, b, Q, TOL_FP32)
        assert r.outcome == CORRECTED and list(np.flatnonzero(r.flagged)) == [2, 11]


def test_full_pipeline_with_additive_errors_decodes_correctly():
    code = GPCode(16, 24, 8, 2, 3, 2, 1, 17)                 # Q_f = 14, corrects up to 2 nodes
    rng = np.random.default_rng(11)
    W, X = rng.standard_normal((16, 24)), rng.standard_normal((24, 8))
    Z = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    nodes = np.zeros(17, dtype=bool)
    nodes[[4, 12]] = True
    inj.inject_additive(Z, seed=12, scale=1.0, nodes=nodes)
    r = locate_subspace(Z, code.points, code.Q_f, TOL_FP64)
    assert r.outcome == CORRECTED and np.array_equal(r.flagged, nodes)
    assert op.rel_fro(op.decode(Z, code, FWD, use=~r.flagged), W @ X) < 1e-8
    # decoding without excluding them is visibly wrong
    assert op.rel_fro(op.decode(Z, code, FWD), W @ X) > 1e-3


def test_injectors_are_reproducible_and_touch_only_selected_nodes():
    Z0 = np.random.default_rng(13).standard_normal((12, 5, 7))
    for fn in (inj.inject_additive, inj.inject_gauss):
        A, Bm = Z0.copy(), Z0.copy()
        sa = fn(A, 99, 2.0, prob=0.3)
        sb = fn(Bm, 99, 2.0, prob=0.3)
        assert np.array_equal(A, Bm) and np.array_equal(sa, sb)
        assert np.array_equal(sa, inj.select_nodes(99, 12, 0.3))
        assert np.array_equal(A[~sa], Z0[~sa])
        assert all((A[p] != Z0[p]).any() for p in np.flatnonzero(sa))
    G = np.zeros((4, 200000))
    inj.inject_gauss(G, 5, 1.0, nodes=[True] * 4)
    assert abs(G.mean()) < 0.01 and abs(G.std() - 1.0) < 0.01
    A = np.zeros((3, 100000))
    inj.inject_additive(A, 6, 1.0, nodes=[True, True, True])
    nz = np.abs(A[A != 0])
    assert nz.min() >= 2.0 ** -4 and nz.max() < 2.0 ** 8
