"""Per-codeword error correction under the adversarial model (test oracle; FP64, numpy).

The lemma on real-number error correction under the adversarial model states that a (P, Q) MDS
code corrects floor((P - Q) / 2) errors of arbitrary value in one codeword: with H the parity
check (H G^T = 0) and z = G^T q + e, the system H e = H z has a unique solution with at most
floor((P - Q) / 2) non-zeros.  The section on decoding methods asks for the solution of H e = H z
with the fewest non-zeros.  Here that is applied to every output position on its own (one codeword
= the P values the nodes hold at that position), so different positions may blame different
nodes - the case the node-level locator of locate.py cannot serve once more than P - Q - 1 nodes
are hit somewhere.

This file is the definition written out: for every position whose syndrome fails the zero test,
supports are tried by increasing size (1 .. t, t = floor((P - Q) / 2)), in lexicographic order
within a size; the first support A with the syndrome in span(H_A) (up to the tolerance) is taken,
the error values are the least-squares solution of H_A e_A = H z, and they are subtracted.

Readings where the paper is silent: the zero tolerance (the same relative test as locate.py,
||r||^2 <= tau_col^2 ||z||^2 with r the syndrome, resp. the part of it outside span(H_A)); a
position holding a non-finite value, or one of magnitude >= 2^500 (its square leaves the FP64 range),
is reported as failed and left untouched; a position that no
support of size <= t explains is reported as failed and left untouched.
"""

from __future__ import annotations

import itertools
from dataclasses import dataclass

import numpy as np

from .code import parity_check
from .locate import CORRECTED, DECODE_FAILURE, HUGE, NO_ERROR, Tolerances


@dataclass
class PositionResult:
    outcome: int                  # NO_ERROR, CORRECTED (every active position repaired), DECODE_FAILURE
    corrected: np.ndarray         # [P, L] outputs with the located errors subtracted
    n_active: int                 # positions that failed the zero test (non-finite ones included)
    n_corrected: int              # of those, repaired
    n_failed: int                 # of those, left untouched
    n_entries: int                # entries changed (sum of support sizes)
    max_errors: int               # largest accepted support
    touched: np.ndarray           # bool[P]: nodes with at least one changed entry
    errors_at: np.ndarray         # int[L]: accepted support size per position (-1 = failed, 0 = clean)


def correct_positions(outputs: np.ndarray, points: np.ndarray, Q: int, tol: Tolerances) -> PositionResult:
    """outputs: [P, L] (any float dtype); arithmetic in FP64."""
    Z = np.array(outputs, dtype=np.float64).reshape(outputs.shape[0], -1)
    P, L = Z.shape
    H = parity_check(np.asarray(points, dtype=np.float64), Q)        # [R, P], orthonormal rows
    R = H.shape[0]
    t = R // 2
    with np.errstate(invalid="ignore"):
        finite = (np.abs(Z) < HUGE).all(axis=0)   # NaN, Inf and values whose square overflows FP64
    Zf = np.where(finite[None, :], Z, 0.0)
    S = H @ Zf                                                        # syndromes, one column per position
    z2 = (Zf ** 2).sum(axis=0)
    limit = tol.tau_col ** 2 * z2
    active = ((S ** 2).sum(axis=0) > limit) | ~finite
    errors_at = np.zeros(L, dtype=np.int64)
    errors_at[active] = -1
    corrected = Z.copy()
    touched = np.zeros(P, dtype=bool)
    n_entries = 0
    todo = np.flatnonzero(active & finite)
    for size in range(1, t + 1):
        for nodes in itertools.combinations(range(P), size):
            if todo.size == 0:
                break
            HA = H[:, nodes]                                          # [R, size]
            coef, *_ = np.linalg.lstsq(HA, S[:, todo], rcond=None)    # least-squares error values
            resid = S[:, todo] - HA @ coef
            ok = (resid ** 2).sum(axis=0) <= limit[todo]
            if ok.any():
                cols = todo[ok]
                corrected[np.ix_(nodes, cols)] -= coef[:, ok]
                errors_at[cols] = size
                touched[list(nodes)] = True
                n_entries += size * cols.size
                todo = todo[~ok]
    n_active = int(active.sum())
    n_failed = int((errors_at < 0).sum())
    outcome = NO_ERROR if n_active == 0 else (DECODE_FAILURE if n_failed else CORRECTED)
    return PositionResult(outcome=outcome, corrected=corrected.reshape(outputs.shape), n_active=n_active,
                          n_corrected=n_active - n_failed, n_failed=n_failed, n_entries=n_entries,
                          max_errors=int(errors_at.max(initial=0)), touched=touched, errors_at=errors_at)
