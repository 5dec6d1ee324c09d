"""Code construction of Generalized PolyDot codes (test oracle; FP64, numpy).

Follows Section IV (Theorems 1 and 2), the DNN versions of Sections VI and VIII
and the single-variable forms in the proofs of Theorems 4 and 6 (appendix on
error tolerances), with the substitution u = v^n, w = v^{mn}.

With the default substitution everything below is a polynomial in the single
variable v evaluated at the node's point b_p:

    W block (i,j)         -> exponent n*i + j                      (Eq. 1 with u=v^n)
    X block (j,k)         -> exponent (n-1-j) + m*n*k              (Theorem 2 encoding, w=v^{mn})
    wanted S block (i,k)  -> exponent n*i + m*n*k + n - 1          (Theorem 2 proof)
    Delta^T block (k,i)   -> exponent m*n*k + n*(m-1-i)            (backpropagation encoding)
    wanted C^T block (k,j)-> exponent m*n*k + n*(m-1) + j          (proof of Theorem 6)
    update operands       -> Delta_i at n*i, X_j at j (ascending)  (update stage)

The alternate substitution v = u^m, w = u^{mn} (second rows of Tables I and III; proofs of
Theorems 4 and 6) makes everything a polynomial in u instead and trades forward for backward
error tolerance:

    W block (i,j) -> i + m*j            X block (j,k) -> m*(n-1-j) + m*n*k
    wanted S (i,k) -> i + m*(n-1) + m*n*k           Q_f = m n d1 + m n - m
    Delta^T block (k,i) -> m*n*k + (m-1-i)          wanted C^T (k,j) -> m*n*k + (m-1) + m*j
    Q_b = m n d2 + m - 1                            update operands: Delta_i at i, X_j at m*j
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

FWD, BWD, UPD, AUDIT = 0, 1, 2, 3
SUBST_U_VN, SUBST_V_UM = 0, 1          # u = v^n, w = v^{mn}   |   v = u^m, w = u^{mn}


def chebyshev_points(P: int) -> np.ndarray:
    """Evaluation points: roots of the first-kind Chebyshev polynomial T_P on [-1,1].

    The paper only asks for P distinct reals; the workloads fix Chebyshev nodes."""
    p = np.arange(P, dtype=np.float64)
    return np.cos((2.0 * p + 1.0) * np.pi / (2.0 * P))


def powers(points: np.ndarray, count: int) -> np.ndarray:
    """V[p, e] = b_p ** e for e = 0..count-1 by repeated multiplication (Vandermonde matrix G^T)."""
    points = np.asarray(points, dtype=np.float64)
    V = np.empty((points.size, count), dtype=np.float64)
    V[:, 0] = 1.0
    for e in range(1, count):
        V[:, e] = V[:, e - 1] * points
    return V


@dataclass
class GPCode:
    """Parameters of one Generalized PolyDot code for a layer W (N1 x N0) and batch B."""

    N1: int
    N0: int
    B: int
    m: int
    n: int
    d1: int = 1
    d2: int = 1
    P: int = 0
    points: Optional[np.ndarray] = None
    subst: int = SUBST_U_VN

    def __post_init__(self):
        if self.N1 % self.m or self.N0 % self.n or self.B % self.d1 or self.B % self.d2:
            raise ValueError("splits must divide the matrix dimensions")
        if self.points is None:
            self.points = chebyshev_points(self.P)
        self.points = np.asarray(self.points, dtype=np.float64)
        if self.points.size != self.P:
            raise ValueError("need exactly P evaluation points")
        if len(set(self.points.tolist())) != self.P:
            raise ValueError("evaluation points must be distinct")

    # ---- recovery thresholds -------------------------------------------------
    @property
    def Q_f(self) -> int:
        """Theorem 2: number of coefficients of S~(v), m n d1 + n - 1 (alternate: m n d1 + m n - m)."""
        if self.subst == SUBST_V_UM:
            return self.m * self.n * self.d1 + self.m * self.n - self.m
        return self.m * self.n * self.d1 + self.n - 1

    @property
    def Q_b(self) -> int:
        """Backpropagation polynomial C~^T(v): m n d2 + m n - n coefficients (alternate: m n d2 + m - 1)."""
        if self.subst == SUBST_V_UM:
            return self.m * self.n * self.d2 + self.m - 1
        return self.m * self.n * (self.d2 + 1) - self.n

    @property
    def Q_w(self) -> int:
        """The stored share W~_p is itself a polynomial of degree mn-1 in v."""
        return self.m * self.n

    def Q(self, which: int) -> int:
        return {FWD: self.Q_f, BWD: self.Q_b, AUDIT: self.Q_w}[which]

    # ---- exponent maps ---------------------------------------------------------
    def exp_W(self) -> np.ndarray:
        i = np.arange(self.m)[:, None]
        j = np.arange(self.n)[None, :]
        if self.subst == SUBST_V_UM:
            return i + self.m * j
        return self.n * i + j                                   # [m, n]

    def exp_X(self) -> np.ndarray:
        j = np.arange(self.n)[:, None]
        k = np.arange(self.d1)[None, :]
        if self.subst == SUBST_V_UM:
            return self.m * (self.n - 1 - j) + self.m * self.n * k
        return (self.n - 1 - j) + self.m * self.n * k           # [n, d1]

    def exp_DeltaT(self) -> np.ndarray:
        k = np.arange(self.d2)[:, None]
        i = np.arange(self.m)[None, :]
        if self.subst == SUBST_V_UM:
            return self.m * self.n * k + (self.m - 1 - i)
        return self.m * self.n * k + self.n * (self.m - 1 - i)  # [d2, m]

    def exp_update(self):
        """Exponents of the ascending update-stage encodings: (Delta_i, X_j)."""
        i, j = np.arange(self.m), np.arange(self.n)
        if self.subst == SUBST_V_UM:
            return i, self.m * j
        return self.n * i, j

    def wanted(self, which: int) -> np.ndarray:
        """Exponent whose coefficient is block (row, col) of the result."""
        if which == FWD:
            i = np.arange(self.m)[:, None]
            k = np.arange(self.d1)[None, :]
            if self.subst == SUBST_V_UM:
                return i + self.m * (self.n - 1) + self.m * self.n * k
            return self.n * i + self.m * self.n * k + self.n - 1      # [m, d1]
        if which == BWD:
            k = np.arange(self.d2)[:, None]
            j = np.arange(self.n)[None, :]
            if self.subst == SUBST_V_UM:
                return self.m * self.n * k + (self.m - 1) + self.m * j
            return self.m * self.n * k + self.n * (self.m - 1) + j    # [d2, n]
        if which == AUDIT:
            return self.exp_W()                                       # [m, n]
        raise ValueError(which)

    # ---- shapes ------------------------------------------------------------------
    def out_block_shape(self, which: int):
        """Shape of one worker output (= one block of the decoded result)."""
        if which == FWD:
            return (self.N1 // self.m, self.B // self.d1)
        if which == BWD:
            return (self.B // self.d2, self.N0 // self.n)
        if which == AUDIT:
            return (self.N1 // self.m, self.N0 // self.n)
        raise ValueError(which)

    # ---- matrices of the (P, Q) real-number MDS code -------------------------------
    def vandermonde(self, Q: int) -> np.ndarray:
        return powers(self.points, Q)


def parity_check(points: np.ndarray, Q: int) -> np.ndarray:
    """H ((P-Q) x P, orthonormal rows) with H G^T = 0 for G^T = Vandermonde(points, Q).

    Rows span the left null space of G^T: the last P-Q columns of the full
    orthogonal factor of a QR factorisation of G^T (Section V-A: parity-check
    matrix of the (P,Q) MDS code)."""
    V = powers(points, Q)
    P = V.shape[0]
    if P <= Q:
        return np.zeros((0, P))
    Qfull, _ = np.linalg.qr(V, mode="complete")
    return np.ascontiguousarray(Qfull[:, Q:].T)
