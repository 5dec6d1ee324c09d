"""Error detection and location over the P worker outputs (test oracle; FP64, numpy).

The paper's Algorithm 1 works on one codeword z (the P values found at one output
position):  (1) if H z = 0 declare "no errors";  (2) else find the sparsest e with
H e = H z;  (3) accept it if it has at most P-Q-1 non-zeros, else declare a
"decoding failure".  Its error models corrupt *whole node outputs*, its tolerances
count *nodes*, and the nodes exchange one length-P vector of "erroneous" flags, so
the decision is taken here at node level, jointly over all L output positions:

  * every column z_l (one codeword) gets Algorithm 1's zero test, in floating point
    ||H z_l||^2 <= tau_col^2 ||z_l||^2  (H has orthonormal rows);
  * the columns that fail it ("active") share one error support A (a set of nodes):
    with Sigma = H Z restricted to the active columns, each normalised by ||z_l||,
    the sparsest consistent support is the smallest A with Sigma in span(H_A).

Two forms are given.  ``locate_exhaustive`` is that definition written out (all
supports by increasing size, lexicographic order).  ``locate_subspace`` is the
polynomial-time form the CUDA library mirrors: since any P-Q columns of H are
independent (MDS property), for |A| <= P-Q-1 and an error matrix of full row rank
(probability 1 under Error Model 2) the column space of Sigma equals span(H_A) and
no other column of H lies in it, so A = {p : H_p in range(Sigma)}.

When the error matrix is rank deficient (errors of several nodes confined to fewer
codewords than nodes, e.g. two bit flips at one output position) fewer columns of H
lie in range(Sigma) than its rank; those that do still belong to A, so the subspace
form then falls back to Algorithm 1's search restricted to supersets of them, by
increasing size, as long as the number of supports tried stays within
``MAX_FALLBACK_SUPPORTS``.

Readings where the paper is silent: the zero tolerances; non-finite values, values of
magnitude >= ``HUGE`` (their squares leave the FP64 range, so no norm test can be
applied to them) and caller-declared erasures are replaced by zero and their node
flagged up front (an erasure is an error of known location and counts against the
P-Q-1 budget); the bound on the fallback search.
"""

from __future__ import annotations

import itertools
import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from .code import parity_check

NO_ERROR, CORRECTED, DECODE_FAILURE = 0, 1, 2
HUGE = 2.0 ** 500                 # |value| >= HUGE is handled like a non-finite value
MAX_FALLBACK_SUPPORTS = 4096      # supports the fallback search of the subspace form may try


@dataclass(frozen=True)
class Tolerances:
    """Zero tests in floating point (engineering constants; not in the paper)."""

    tau_col: float   # a codeword's syndrome is zero if ||H z|| <= tau_col * ||z||
    tau_in: float    # a node is inside the error subspace if its distance is <= tau_in


# FP32 outputs: rounding and FP32 accumulation leave a clean-syndrome floor near 1e-6 of ||z||;
# FP64 outputs: the floor is near 1e-15, but the Gram matrix of syndromes only resolves energy
# ratios down to about 2^-44, so the tolerance is kept at 2^-20 (energy 2^-40).
TOL_FP32 = Tolerances(tau_col=2.0 ** -13, tau_in=2.0 ** -15)   # worker outputs stored in FP32
TOL_FP64 = Tolerances(tau_col=2.0 ** -20, tau_in=2.0 ** -30)   # worker outputs stored in FP64


def tolerances_for(dtype) -> Tolerances:
    return TOL_FP32 if np.dtype(dtype) == np.float32 else TOL_FP64


@dataclass
class LocateResult:
    outcome: int
    flagged: np.ndarray                       # bool[P]: nodes whose output must not be used
    n_active: int = 0                         # codewords that failed the zero test
    rank: int = 0                             # numerical rank of the syndrome Gram matrix
    residual: float = 0.0                     # tr((I - Pi_A) G) / n_active for the accepted A
    forced: np.ndarray = field(default=None)  # bool[P]: erased or non-finite nodes

    @property
    def n_flagged(self) -> int:
        return int(self.flagged.sum())


def syndrome_gram(outputs: np.ndarray, H: np.ndarray, tol: Tolerances,
                  erased: Optional[Sequence[bool]] = None):
    """Step 1 of Algorithm 1 on every codeword, and the Gram matrix of the failing ones.

    Returns (G, n_active, forced).  outputs: [P, L] (any float dtype)."""
    P = outputs.shape[0]
    Z = np.asarray(outputs, dtype=np.float64).reshape(P, -1).copy()
    er = np.zeros(P, dtype=bool) if erased is None else np.asarray(erased, dtype=bool)
    with np.errstate(invalid="ignore"):
        finite = np.abs(Z) < HUGE     # False for NaN, Inf and for values whose square overflows
    forced = er | ~finite.all(axis=1)
    Z[~finite] = 0.0          # a non-finite value is replaced by zero, its node flagged
    Z[er, :] = 0.0            # an erased node contributes nothing
    Sigma = H @ Z                                         # (P-Q) x L
    ns = np.einsum("rl,rl->l", Sigma, Sigma)
    nz = np.einsum("pl,pl->l", Z, Z)
    active = (nz > 0.0) & (ns > tol.tau_col ** 2 * nz)
    Sa = Sigma[:, active] / np.sqrt(nz[active])[None, :]
    G = Sa @ Sa.T
    return G, int(active.sum()), forced


def _residual(G: np.ndarray, H: np.ndarray, nodes: Sequence[int]) -> float:
    """tr((I - Pi) G (I - Pi)) with Pi the orthogonal projector on span(H[:, nodes])."""
    if len(nodes) == 0:
        return float(np.trace(G))
    Qa, _ = np.linalg.qr(H[:, list(nodes)])
    Pi = Qa @ Qa.T
    I = np.eye(H.shape[0])
    return float(np.trace((I - Pi) @ G @ (I - Pi)))


def locate_exhaustive(outputs: np.ndarray, points: np.ndarray, Q: int, tol: Tolerances,
                      erased: Optional[Sequence[bool]] = None) -> LocateResult:
    """Algorithm 1 at node level, by brute force: supports by increasing size, lexicographic."""
    P = outputs.shape[0]
    H = parity_check(points, Q)
    G, n_active, forced = syndrome_gram(outputs, H, tol, erased)
    forced_idx = [int(p) for p in np.flatnonzero(forced)]
    budget = P - Q - 1
    if n_active == 0 and not forced_idx:
        return LocateResult(NO_ERROR, np.zeros(P, dtype=bool), 0, 0, 0.0, forced)
    limit = tol.tau_col ** 2 * max(n_active, 1)
    free = [p for p in range(P) if p not in forced_idx]
    for size in range(len(forced_idx), budget + 1):
        best, best_set = None, None
        for extra in itertools.combinations(free, size - len(forced_idx)):
            nodes = sorted(forced_idx + list(extra))
            r = _residual(G, H, nodes)
            if best is None or r < best:
                best, best_set = r, nodes
        if best is not None and best <= limit:
            flagged = np.zeros(P, dtype=bool)
            flagged[best_set] = True
            return LocateResult(CORRECTED, flagged, n_active, size, best / max(n_active, 1), forced)
    flagged = forced.copy()
    return LocateResult(DECODE_FAILURE, flagged, n_active, 0, 0.0, forced)


def _superset_search(G: np.ndarray, H: np.ndarray, base: np.ndarray, budget: int, n_active: int,
                     rank: int, tol: Tolerances, forced: np.ndarray) -> LocateResult:
    """Algorithm 1's search over the supports that contain ``base`` (nodes already known to be
    erroneous): sizes in increasing order, lexicographic within a size, the first support whose
    residual passes is taken.  A size is searched only while the running number of supports
    stays within MAX_FALLBACK_SUPPORTS; otherwise a decoding failure is declared."""
    P = H.shape[1]
    base_idx = [int(p) for p in np.flatnonzero(base)]
    free = [p for p in range(P) if not base[p]]
    limit = tol.tau_col ** 2 * max(n_active, 1)
    tried = 0
    for size in range(len(base_idx), budget + 1):
        extra_n = size - len(base_idx)
        tried += math.comb(len(free), extra_n)
        if tried > MAX_FALLBACK_SUPPORTS:
            break
        for extra in itertools.combinations(free, extra_n):
            nodes = sorted(base_idx + list(extra))
            r = _residual(G, H, nodes)
            if r <= limit:
                flagged = np.zeros(P, dtype=bool)
                flagged[nodes] = True
                return LocateResult(CORRECTED, flagged, n_active, rank, r / max(n_active, 1), forced)
    return LocateResult(DECODE_FAILURE, forced.copy(), n_active, rank, 0.0, forced)


def locate_subspace(outputs: np.ndarray, points: np.ndarray, Q: int, tol: Tolerances,
                    erased: Optional[Sequence[bool]] = None) -> LocateResult:
    """Polynomial-time form: eigen-decompose the syndrome Gram matrix, read the support off
    the columns of H that lie in its range, then verify the residual."""
    P = outputs.shape[0]
    H = parity_check(points, Q)
    R = P - Q
    G, n_active, forced = syndrome_gram(outputs, H, tol, erased)
    budget = R - 1
    if n_active == 0 and not forced.any():
        return LocateResult(NO_ERROR, np.zeros(P, dtype=bool), 0, 0, 0.0, forced)
    if forced.sum() > budget:
        return LocateResult(DECODE_FAILURE, forced.copy(), n_active, 0, 0.0, forced)
    flagged = forced.copy()
    rank = 0
    if n_active > 0:
        lam, U = np.linalg.eigh(G)
        lam, U = lam[::-1], U[:, ::-1]
        theta = tol.tau_col ** 2 * n_active / R
        rank = int((lam > theta).sum())
        if rank > budget:
            return LocateResult(DECODE_FAILURE, forced.copy(), n_active, rank, 0.0, forced)
        Ur = U[:, :rank]
        resid = H - Ur @ (Ur.T @ H)                        # component of each H_p outside range(G)
        dist = np.linalg.norm(resid, axis=0) / np.linalg.norm(H, axis=0)
        inside = dist <= tol.tau_in
        flagged |= inside
        if int(inside.sum()) != rank:                      # rank-deficient error matrix
            return _superset_search(G, H, flagged, budget, n_active, rank, tol, forced)
    if flagged.sum() > budget:
        return LocateResult(DECODE_FAILURE, forced.copy(), n_active, rank, 0.0, forced)
    r = _residual(G, H, np.flatnonzero(flagged))
    if r > tol.tau_col ** 2 * max(n_active, 1):
        return LocateResult(DECODE_FAILURE, forced.copy(), n_active, rank, 0.0, forced)
    return LocateResult(CORRECTED, flagged, n_active, rank, r / max(n_active, 1), forced)
