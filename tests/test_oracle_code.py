"""Pins of the oracle's code construction, encoding and decoding against the paper and the maths."""

import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle.code import GPCode, FWD, BWD, AUDIT, chebyshev_points, parity_check, powers
from oracle import product as op
import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kv(path):
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, *v = line.split()
            out[k] = [int(x) for x in v]
    return out


def test_worked_example_printed_numbers():
    g = _kv(os.path.join(GOLDEN, "worked_example_2x2x2.txt"))
    m, n, d = g["m"][0], g["n"][0], g["d"][0]
    code = GPCode(N1=4, N0=4, B=4, m=m, n=n, d1=d, P=11)
    w = code.wanted(FWD)
    for i in range(m):
        for k in range(d):
            assert w[i, k] == g[f"wanted_exponent_i{i}_k{k}"][0]
    assert code.Q_f == g["threshold"][0]
    assert code.Q_f - 1 == g["degree"][0]
    # the unaligned trivariate polynomial has m * (2n-1) * d coefficients
    assert m * (2 * n - 1) * d == g["unaligned_coefficients"][0]


def test_chebyshev_points_are_the_roots_of_T_P():
    """Evaluation points of the workloads: the P roots of the first-kind Chebyshev polynomial,
    in decreasing order (closed forms for P = 1, 2, 3; T_P(b_p) = 0 through numpy's Chebyshev
    series evaluation; the extrema of T_P, the second-kind points, would fail every line)."""
    assert np.allclose(chebyshev_points(1), [0.0], atol=1e-16)
    assert np.allclose(chebyshev_points(2), [np.sqrt(0.5), -np.sqrt(0.5)], rtol=0, atol=1e-15)
    assert np.allclose(chebyshev_points(3), [np.sqrt(3) / 2, 0.0, -np.sqrt(3) / 2], rtol=0, atol=1e-15)
    for P in (2, 3, 10, 11, 13, 25, 36, 40, 64):
        b = chebyshev_points(P)
        assert b.shape == (P,) and np.all(np.diff(b) < 0) and np.all(np.abs(b) < 1)
        T_P = np.zeros(P + 1)
        T_P[P] = 1.0
        assert np.abs(np.polynomial.chebyshev.chebval(b, T_P)).max() < 1e-13 * P
        assert np.allclose(b, -b[::-1], rtol=0, atol=1e-15)          # symmetric about zero
        # the P roots of the degree-P monic polynomial 2^(1-P) T_P: their product is its constant term
        if P % 2 == 0:
            assert np.isclose(np.prod(b), (-1) ** (P // 2) * 2.0 ** (1 - P), rtol=1e-12)


def test_printed_thresholds():
    for line in open(os.path.join(GOLDEN, "printed_thresholds.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        m, n, d, thr = (int(x) for x in line.split())
        code = GPCode(N1=m, N0=n, B=d, m=m, n=n, d1=d, P=thr + 1)
        assert code.Q_f == thr


@pytest.mark.parametrize("m,n,d", [(m, n, d) for m in range(1, 5) for n in range(1, 5) for d in range(1, 5)])
def test_thresholds_by_brute_force_exponent_count(m, n, d):
    """Expand W~(v) X~(v) and Delta~^T(v) W~(v) term by term; count distinct exponents and check
    that a wanted exponent only ever receives the terms that make up its block."""
    code = GPCode(N1=m, N0=n, B=d, m=m, n=n, d1=d, d2=d, P=64,
                  points=np.linspace(-1, 1, 64))
    eW, eX, eD = code.exp_W(), code.exp_X(), code.exp_DeltaT()
    # forward
    terms = {}
    for i, j, jp, k in itertools.product(range(m), range(n), range(n), range(d)):
        terms.setdefault(int(eW[i, j] + eX[jp, k]), []).append((i, j, jp, k))
    assert max(terms) + 1 == code.Q_f == m * n * d + n - 1          # Theorem 2
    assert len(terms) <= code.Q_f
    want = code.wanted(FWD)
    for i, k in itertools.product(range(m), range(d)):
        got = sorted(terms[int(want[i, k])])
        assert got == [(i, j, j, k) for j in range(n)]              # exactly S_ik = sum_j W_ij X_jk
    # backward
    terms = {}
    for k, ip, i, j in itertools.product(range(d), range(m), range(m), range(n)):
        terms.setdefault(int(eD[k, ip] + eW[i, j]), []).append((k, ip, i, j))
    assert max(terms) + 1 == code.Q_b == m * n * (d + 1) - n
    want = code.wanted(BWD)
    for k, j in itertools.product(range(d), range(n)):
        assert sorted(terms[int(want[k, j])]) == [(k, i, i, j) for i in range(m)]
    # the share itself
    assert sorted(eW.reshape(-1).tolist()) == list(range(m * n)) and code.Q_w == m * n


def test_workload_node_counts_are_threshold_plus_extra():
    c1, c2, c3 = wl.CONFIG_1_TINY, wl.CONFIG_2_MATVEC, wl.CONFIG_3_MATMUL
    for c, extra in ((c1, 2), (c2, 4), (c3, 6)):
        code = GPCode(c.N1, c.N0, c.B, c.m, c.n, c.d, 1, c.P)
        assert c.P == code.Q_f + extra
    c4 = wl.CONFIG_4_MLP
    code = GPCode(c4.widths[1], c4.widths[0], c4.B, c4.m, c4.n, c4.d1, c4.d2, c4.P)
    assert (code.Q_f, code.Q_b, code.Q_w) == (5, 6, 4) and c4.P == max(code.Q_f, code.Q_b) + 4
    c5 = wl.CONFIG_5_AUTOENCODER
    code = GPCode(c5.n_hidden, c5.n_visible, c5.B, c5.m, c5.n, c5.d1, c5.d2, c5.P)
    assert (code.Q_f, code.Q_b, code.Q_w) == (19, 28, 16) and c5.P == max(code.Q_f, code.Q_b) + 8


def test_error_tolerance_tables():
    """Tables I and III, Generalized PolyDot row with u = v^n: (t_f, t_b) under both models."""
    for (m, n, d1, d2, P) in [(6, 6, 1, 1, 180), (2, 2, 1, 1, 10), (4, 4, 1, 1, 36), (2, 4, 2, 3, 60)]:
        code = GPCode(m * 2, n * 2, d1 * d2 * 2, m, n, d1, d2, P)
        assert P - code.Q_f == P - d1 * m * n - n + 1                 # P - Q = 2 t_f (+1) under Model 1
        assert (P - code.Q_f) // 2 == (P - d1 * m * n - n + 1) // 2
        assert P - code.Q_f - 1 == P - d1 * m * n - n                 # Model 2
        assert (P - code.Q_b) // 2 == (P - (d2 + 1) * m * n + n) // 2
        assert P - code.Q_b - 1 == P - (d2 + 1) * m * n + n - 1
    # values at the parameters of the tolerance-region figure (P = 180, m = n = 6)
    code = GPCode(6, 6, 1, 6, 6, 1, 1, 180)
    assert ((180 - code.Q_f) // 2, (180 - code.Q_b) // 2) == (69, 57)
    assert (180 - code.Q_f - 1, 180 - code.Q_b - 1) == (138, 113)


# ----------------------------------------------------------------------------------------------
# encoding
# ----------------------------------------------------------------------------------------------
def _rand(shape, seed):
    return np.random.default_rng(seed).uniform(-1, 1, size=shape)


def test_encode_special_cases():
    W, X = _rand((6, 8), 0), _rand((8, 4), 1)
    # one block: the share is the input at every node
    code = GPCode(6, 8, 4, 1, 1, 1, 1, 3)
    assert np.array_equal(op.encode_W(W, code), np.broadcast_to(W, (3, 6, 8)))
    assert np.array_equal(op.encode_X(X, code), np.broadcast_to(X, (3, 8, 4)))
    # points 0 and 1: constant term alone / plain sum of blocks
    code = GPCode(6, 8, 4, 3, 2, 2, 2, 3, points=np.array([0.0, 1.0, -1.0]))
    Ws, Xs, Ds = op.encode_W(W, code), op.encode_X(X, code), op.encode_DeltaT(_rand((4, 6), 2), code)
    assert np.array_equal(Ws[0], W[:2, :4])                                  # W_00
    assert np.array_equal(Xs[0], X[4:, :2])                                  # X_{n-1,0}
    assert np.allclose(Ws[1], sum(W[2 * i:2 * i + 2, 4 * j:4 * j + 4] for i in range(3) for j in range(2)))
    assert np.allclose(Xs[1], sum(X[4 * j:4 * j + 4, 2 * k:2 * k + 2] for j in range(2) for k in range(2)))
    D = _rand((4, 6), 2)
    assert np.array_equal(Ds[0], D[:2, 4:])                                  # Delta^T_{0, m-1}
    # point -1: signs follow the exponent's parity
    sg = (-1.0) ** code.exp_W()
    assert np.allclose(Ws[2], sum(sg[i, j] * W[2 * i:2 * i + 2, 4 * j:4 * j + 4] for i in range(3) for j in range(2)))


def test_encode_is_linear_and_matches_polynomial_evaluation():
    code = GPCode(8, 6, 4, 2, 3, 2, 1, 7)
    A, Bm = _rand((8, 6), 3), _rand((8, 6), 4)
    assert np.allclose(op.encode_W(2 * A - 3 * Bm, code), 2 * op.encode_W(A, code) - 3 * op.encode_W(Bm, code))
    # entry (r,c) of share p is the polynomial sum_ij W_ij[r,c] v^(n i + j) evaluated at b_p (np.polyval)
    sh = op.encode_W(A, code)
    coeffs = np.zeros(code.Q_w)
    for i in range(2):
        for j in range(3):
            coeffs[3 * i + j] = A[4 * i + 1, 2 * j + 1]
    for p in range(code.P):
        assert np.isclose(sh[p, 1, 1], np.polyval(coeffs[::-1], code.points[p]), rtol=1e-13)


# ----------------------------------------------------------------------------------------------
# decoding
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,n,d,P", [(2, 2, 2, 11), (4, 2, 1, 13), (1, 4, 1, 9), (3, 1, 3, 10), (2, 3, 2, 16)])
def test_decoded_equals_uncoded_forward_backward_audit(m, n, d, P):
    N1, N0, B = 4 * m, 6 * n, 2 * d
    code = GPCode(N1, N0, B, m, n, d, d, P)
    if P < max(code.Q_f, code.Q_b):
        code = GPCode(N1, N0, B, m, n, d, d, max(code.Q_f, code.Q_b) + 2)
    W, X, DT = _rand((N1, N0), 5), _rand((N0, B), 6), _rand((B, N1), 7)
    Ws = op.encode_W(W, code)
    S = op.decode(op.worker_products(Ws, op.encode_X(X, code)), code, FWD)
    assert op.rel_fro(S, W @ X) < 1e-9
    CT = op.decode(op.worker_products(op.encode_DeltaT(DT, code), Ws), code, BWD)
    assert op.rel_fro(CT, DT @ W) < 1e-7
    assert op.rel_fro(op.decode(Ws, code, AUDIT), W) < 1e-10


def test_config1_every_threshold_sized_subset_decodes_the_same():
    cfg = wl.CONFIG_1_TINY
    W, X = wl.matmul_inputs(cfg)
    code = GPCode(cfg.N1, cfg.N0, cfg.B, cfg.m, cfg.n, cfg.d, 1, cfg.P)
    Z = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    ref = op.ref_forward(W, X)
    n_sub = 0
    for keep in itertools.combinations(range(cfg.P), code.Q_f):
        use = np.zeros(cfg.P, dtype=bool)
        use[list(keep)] = True
        assert op.rel_fro(op.decode(Z, code, FWD, use), ref) < 1e-7
        n_sub += 1
    assert n_sub == 55


def test_decode_exact_rational_lagrange():
    """Integer inputs, rational points: the wanted coefficients obtained by exact Lagrange
    interpolation (python fractions) equal W X exactly, and the FP64 decode agrees."""
    m, n, d = 2, 2, 2
    rng = np.random.default_rng(8)
    W = rng.integers(-3, 4, size=(4, 4))
    X = rng.integers(-3, 4, size=(4, 4))
    pts = [Fraction(k, 8) for k in (-7, -5, -3, -2, -1, 1, 2, 4, 6)]            # Q = 9 points
    code = GPCode(4, 4, 4, m, n, d, 1, 9, points=np.array([float(p) for p in pts]))
    Z = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    # exact shares and products
    eW, eX = code.exp_W(), code.exp_X()
    Zx = []
    for b in pts:
        Wt = [[sum(int(W[2 * i + r, 2 * j + c]) * b ** int(eW[i, j]) for i in range(2) for j in range(2))
               for c in range(2)] for r in range(2)]
        Xt = [[sum(int(X[2 * j + r, 2 * k + c]) * b ** int(eX[j, k]) for j in range(2) for k in range(2))
               for c in range(2)] for r in range(2)]
        Zx.append([[sum(Wt[r][t] * Xt[t][c] for t in range(2)) for c in range(2)] for r in range(2)])
    for p in range(9):
        assert np.allclose(Z[p], np.array([[float(v) for v in row] for row in Zx[p]]), rtol=1e-14)

    def lagrange_coeffs(ys):
        """Coefficients (ascending) of the unique degree-8 polynomial through (pts, ys)."""
        total = [Fraction(0)] * 9
        for a, ya in enumerate(ys):
            basis, den = [Fraction(1)], Fraction(1)
            for c, xc in enumerate(pts):
                if c == a:
                    continue
                basis = [(basis[t - 1] if t > 0 else 0) - xc * (basis[t] if t < len(basis) else 0)
                         for t in range(len(basis) + 1)]
                den *= pts[a] - xc
            for t in range(9):
                total[t] += ya * basis[t] / den
        return total

    S_exact = W @ X
    S = op.decode(Z, code, FWD)
    want = code.wanted(FWD)
    for r in range(2):
        for c in range(2):
            co = lagrange_coeffs([Zx[p][r][c] for p in range(9)])
            for i in range(2):
                for k in range(2):
                    assert co[int(want[i, k])] == int(S_exact[2 * i + r, 2 * k + c])
    assert np.allclose(S, S_exact, atol=1e-9)


def test_decode_matrix_matches_decode():
    code = GPCode(8, 8, 4, 2, 2, 2, 1, 12)
    W, X = _rand((8, 8), 9), _rand((8, 4), 10)
    Z = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    use = np.ones(12, dtype=bool)
    use[[1, 7]] = False
    D = op.decode_matrix(code, FWD, use)
    blocks = (D @ Z.reshape(12, -1)).reshape(2, 2, 4, 2)
    S = blocks.transpose(0, 2, 1, 3).reshape(8, 4)
    assert np.allclose(S, op.decode(Z, code, FWD, use), atol=1e-12)
    assert np.all(D[:, ~use] == 0)


def test_update_preserves_the_code():
    """Eq. (10): decoding the updated shares gives W + eta Delta X^T (with weight decay too)."""
    code = GPCode(8, 12, 6, 2, 3, 1, 1, 9)
    W, D, X = _rand((8, 12), 11), _rand((8, 6), 12), _rand((12, 6), 13)
    Dh, Xh = op.encode_update_operands(D, X, code)
    for lam in (0.0, 0.3):
        new = op.update_shares(op.encode_W(W, code), Dh, Xh, eta=0.05, lam=lam)
        assert op.rel_fro(op.decode(new, code, AUDIT), op.ref_update(W, D, X, 0.05, lam)) < 1e-11
        assert np.allclose(new, op.encode_W(op.ref_update(W, D, X, 0.05, lam), code), atol=1e-12)


# ----------------------------------------------------------------------------------------------
# parity-check matrix
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("P,Q", [(11, 9), (13, 9), (25, 19), (10, 5), (36, 28), (36, 16)])
def test_parity_check_annihilates_codewords_and_matches_closed_form(P, Q):
    b = chebyshev_points(P)
    H = parity_check(b, Q)
    V = powers(b, Q)
    assert H.shape == (P - Q, P)
    assert np.abs(H @ V).max() < 1e-13
    assert np.allclose(H @ H.T, np.eye(P - Q), atol=1e-13)
    # closed form: rows b^t * w, t < P-Q, with w_p = 1 / prod_{q != p} (b_p - b_q)  (divided differences
    # of a polynomial of degree < P-1 vanish); the two row spaces must coincide
    w = np.array([1.0 / np.prod([b[p] - b[q] for q in range(P) if q != p]) for p in range(P)])
    C = powers(b, P - Q).T * w[None, :]
    C /= np.linalg.norm(C, axis=1, keepdims=True)
    assert np.abs(C @ V).max() < 1e-9
    proj = H.T @ H
    resid = C - C @ proj
    assert np.abs(resid).max() < 1e-6


def test_parity_check_is_mds_on_small_codes():
    """Any P-Q columns of H are linearly independent (H generates a (P, P-Q) MDS code)."""
    P, Q = 8, 5
    H = parity_check(chebyshev_points(P), Q)
    for cols in itertools.combinations(range(P), P - Q):
        assert np.linalg.svd(H[:, cols], compute_uv=False)[-1] > 1e-6


# ----------------------------------------------------------------------------------------------
# regeneration of erroneous nodes' shares
# ----------------------------------------------------------------------------------------------
def test_regeneration_restores_any_set_of_up_to_P_minus_mn_shares():
    """A share is the evaluation of a degree mn-1 polynomial: whatever was stored at up to P - mn
    nodes, interpolating from the others and re-evaluating gives back the encoding of W."""
    code = GPCode(8, 6, 2, 2, 3, 1, 1, 9)                      # mn = 6: any 3 shares can be lost
    W = _rand((8, 6), 21)
    clean = op.encode_W(W, code)
    rng = np.random.default_rng(22)
    for size in range(0, 4):
        for nodes in itertools.combinations(range(9), size):
            bad = clean.copy()
            flagged = np.zeros(9, dtype=bool)
            flagged[list(nodes)] = True
            bad[flagged] = rng.standard_normal(bad[flagged].shape) * 7
            assert np.allclose(op.regenerate_shares(bad, code, flagged), clean, atol=1e-10)
    # the regenerated value is the polynomial's value: with one block per monomial it is W~(b_p) itself
    flagged = np.zeros(9, dtype=bool)
    flagged[4] = True
    again = op.regenerate_shares(clean, code, flagged)
    coeffs = [W[4 * i + 1, 2 * j + 1] for i in range(2) for j in range(3)]
    assert np.isclose(again[4, 1, 1], np.polyval(coeffs[::-1], code.points[4]), rtol=1e-12)
    with pytest.raises(ValueError):
        op.regenerate_shares(clean, code, np.array([True] * 4 + [False] * 5))


# ----------------------------------------------------------------------------------------------
# alternate substitution v = u^m, w = u^{mn}
# ----------------------------------------------------------------------------------------------
from oracle.code import SUBST_V_UM   # noqa: E402


@pytest.mark.parametrize("m,n,d", [(m, n, d) for m in range(1, 5) for n in range(1, 5) for d in range(1, 4)])
def test_alternate_substitution_thresholds_by_brute_force(m, n, d):
    code = GPCode(m, n, d, m, n, d, d, 64, points=np.linspace(-1, 1, 64), subst=SUBST_V_UM)
    eW, eX, eD = code.exp_W(), code.exp_X(), code.exp_DeltaT()
    terms = {}
    for i, j, jp, k in itertools.product(range(m), range(n), range(n), range(d)):
        terms.setdefault(int(eW[i, j] + eX[jp, k]), []).append((i, j, jp, k))
    assert max(terms) + 1 == code.Q_f == m * n * d + m * n - m            # proof of Theorem 6, second case
    want = code.wanted(FWD)
    for i, k in itertools.product(range(m), range(d)):
        assert sorted(terms[int(want[i, k])]) == [(i, j, j, k) for j in range(n)]
    terms = {}
    for k, ip, i, j in itertools.product(range(d), range(m), range(m), range(n)):
        terms.setdefault(int(eD[k, ip] + eW[i, j]), []).append((k, ip, i, j))
    assert max(terms) + 1 == code.Q_b == m * n * d + m - 1
    want = code.wanted(BWD)
    for k, j in itertools.product(range(d), range(n)):
        assert sorted(terms[int(want[k, j])]) == [(k, i, i, j) for i in range(m)]
    assert sorted(eW.reshape(-1).tolist()) == list(range(m * n))


def test_alternate_substitution_tolerances_and_products():
    # Table I, second row, at P = 180, m = n = 6: (t_f, t_b) swap roles
    code = GPCode(6, 6, 1, 6, 6, 1, 1, 180, subst=SUBST_V_UM)
    assert ((180 - code.Q_f) // 2, (180 - code.Q_b) // 2) == (57, 69)
    assert (180 - code.Q_f - 1, 180 - code.Q_b - 1) == (113, 138)
    code = GPCode(12, 8, 6, 3, 2, 2, 3, 26, subst=SUBST_V_UM)
    W, X, DT = _rand((12, 8), 31), _rand((8, 6), 32), _rand((6, 12), 33)
    Ws = op.encode_W(W, code)
    assert op.rel_fro(op.decode(op.worker_products(Ws, op.encode_X(X, code)), code, FWD), W @ X) < 1e-8
    assert op.rel_fro(op.decode(op.worker_products(op.encode_DeltaT(DT, code), Ws), code, BWD), DT @ W) < 1e-8
    Dh, Xh = op.encode_update_operands(DT.T.copy(), X, code)
    new = op.update_shares(Ws, Dh, Xh, eta=0.1)
    assert op.rel_fro(op.decode(new, code, AUDIT), op.ref_update(W, DT.T, X, 0.1)) < 1e-10
