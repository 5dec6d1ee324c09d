"""Encode / worker products / interpolation decode / coded update (test oracle; FP64, numpy).

Layouts (all row-major, paper orientation):
    W        N1 x N0          W shares        [P][N1/m][N0/n]
    X        N0 x B           X shares        [P][N0/n][B/d1]
    Delta^T  B  x N1          Delta^T shares  [P][B/d2][N1/m]
    S~       [P][N1/m][B/d1]  C~^T            [P][B/d2][N0/n]
"""

from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from .code import GPCode, FWD, BWD, AUDIT, powers


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=np.float64)


# ---------------------------------------------------------------------------------------
# Uncoded reference products (Section II-B: steps O1, O2, O3)
# ---------------------------------------------------------------------------------------
def ref_forward(W, X) -> np.ndarray:
    return _f64(W) @ _f64(X)


def ref_backward(DeltaT, W) -> np.ndarray:
    return _f64(DeltaT) @ _f64(W)


def ref_update(W, Delta, X, eta: float, lam: float = 0.0) -> np.ndarray:
    return (1.0 - eta * lam) * _f64(W) + eta * (_f64(Delta) @ _f64(X).T)


# ---------------------------------------------------------------------------------------
# Encoding (Eq. 1 / Eq. 3 for W; Theorem 2's X~; backpropagation's Delta~^T; update operands)
# ---------------------------------------------------------------------------------------
def _encode_blocks(M: np.ndarray, rows: int, cols: int, exps: np.ndarray, code: GPCode) -> np.ndarray:
    """share_p = sum over blocks (r,c) of b_p ** exps[r,c] * M_block(r,c)."""
    M = _f64(M)
    br, bc = M.shape[0] // rows, M.shape[1] // cols
    pw = powers(code.points, int(exps.max()) + 1)
    out = np.zeros((code.P, br, bc), dtype=np.float64)
    for r in range(rows):
        for c in range(cols):
            blk = M[r * br:(r + 1) * br, c * bc:(c + 1) * bc]
            coef = pw[:, exps[r, c]]
            out += coef[:, None, None] * blk[None, :, :]
    return out


def encode_W(W, code: GPCode) -> np.ndarray:
    """W~_p = sum_ij W_ij a_p^i b_p^j with a_p = b_p^n."""
    return _encode_blocks(W, code.m, code.n, code.exp_W(), code)


def encode_X(X, code: GPCode) -> np.ndarray:
    """X~_p = sum_jk X_jk b_p^{n-1-j} c_p^k with c_p = b_p^{mn}."""
    return _encode_blocks(X, code.n, code.d1, code.exp_X(), code)


def encode_DeltaT(DeltaT, code: GPCode) -> np.ndarray:
    """Delta~^T_p = sum_ki Delta^T_{k,i} c_p^k a_p^{m-1-i}."""
    return _encode_blocks(DeltaT, code.d2, code.m, code.exp_DeltaT(), code)


def encode_update_operands(Delta, X, code: GPCode):
    """Ascending-power encodings of the update stage:
    Delta^_p = sum_i Delta_i a_p^i  ([P][N1/m][B]),  X^_p = sum_j X_j b_p^j  ([P][N0/n][B])."""
    eD, eX = code.exp_update()
    eD, eX = eD[:, None], eX[:, None]
    Dh = _encode_blocks(Delta, code.m, 1, eD, code)
    Xh = _encode_blocks(X, code.n, 1, eX, code)
    return Dh, Xh


# ---------------------------------------------------------------------------------------
# Worker products: node p multiplies its two shares (steps O1, O2) or updates its share (O3)
# ---------------------------------------------------------------------------------------
def worker_products(left_shares: np.ndarray, right_shares: np.ndarray) -> np.ndarray:
    """out[p] = left[p] @ right[p]; forward: (W~, X~); backward: (Delta~^T, W~)."""
    return np.matmul(_f64(left_shares), _f64(right_shares))


def update_shares(W_shares, Dhat, Xhat, eta: float, lam: float = 0.0) -> np.ndarray:
    """W~_p <- (1 - eta*lam) W~_p + eta * Delta^_p X^_p^T  (Eq. 10 and its regularised form)."""
    return (1.0 - eta * lam) * _f64(W_shares) + eta * np.matmul(_f64(Dhat), np.swapaxes(_f64(Xhat), 1, 2))


# ---------------------------------------------------------------------------------------
# Decoding: interpolate the polynomial from the clean evaluations, keep the wanted coefficients
# ---------------------------------------------------------------------------------------
def decode_matrix(code: GPCode, which: int, use: Sequence[bool]) -> np.ndarray:
    """D [n_wanted, P]: rows of the least-squares inverse of the Vandermonde system restricted
    to the nodes in ``use`` (columns of unused nodes are zero).  Row order: row-major over the
    wanted block grid."""
    use = np.asarray(use, dtype=bool)
    Q = code.Q(which)
    if use.sum() < Q:
        raise ValueError("fewer clean nodes than the recovery threshold")
    V = code.vandermonde(Q)[use]                       # |S| x Q
    Qm, R = np.linalg.qr(V)                            # V = Qm R
    pinv = np.linalg.solve(R, Qm.T)                    # Q x |S|
    wanted = code.wanted(which).reshape(-1)
    D = np.zeros((wanted.size, code.P), dtype=np.float64)
    D[:, use] = pinv[wanted, :]
    return D


def decode(outputs: np.ndarray, code: GPCode, which: int, use: Optional[Sequence[bool]] = None) -> np.ndarray:
    """Solve G^T q = z on the clean nodes for every output position and assemble the result
    (S: N1 x B, C^T: B x N0, or W: N1 x N0) from the wanted coefficients."""
    if use is None:
        use = np.ones(code.P, dtype=bool)
    use = np.asarray(use, dtype=bool)
    Q = code.Q(which)
    if use.sum() < Q:
        raise ValueError("fewer clean nodes than the recovery threshold")
    br, bc = code.out_block_shape(which)
    Z = _f64(outputs).reshape(code.P, br * bc)[use]    # |S| x L
    V = code.vandermonde(Q)[use]
    Qm, R = np.linalg.qr(V)
    coeffs = np.linalg.solve(R, Qm.T @ Z)              # Q x L : all coefficients of the polynomial
    wanted = code.wanted(which)
    rows, cols = wanted.shape
    out = np.empty((rows * br, cols * bc), dtype=np.float64)
    for r in range(rows):
        for c in range(cols):
            out[r * br:(r + 1) * br, c * bc:(c + 1) * bc] = coeffs[wanted[r, c]].reshape(br, bc)
    return out


def regenerate_shares(W_shares: np.ndarray, code: GPCode, flagged: Sequence[bool]) -> np.ndarray:
    """Regeneration (Section VI): every share is the evaluation at b_p of the polynomial
    sum_ij W_ij v^(n i + j) of degree mn - 1, so the shares of the flagged nodes are recomputed
    by interpolating that polynomial from the clean nodes (all of them, least squares) and
    evaluating it at the flagged nodes' points.  Only the polynomial's values are needed, not its
    monomial coefficients, so the fit is done in the Chebyshev basis (numpy.polynomial.chebyshev),
    which keeps the system well conditioned on [-1,1].  Returns a new array."""
    flagged = np.asarray(flagged, dtype=bool)
    use = ~flagged
    Q = code.Q_w
    if use.sum() < Q:
        raise ValueError("fewer clean nodes than mn")
    out = _f64(W_shares).copy()
    if not flagged.any():
        return out
    shape = out.shape[1:]
    V = np.polynomial.chebyshev.chebvander(code.points, Q - 1)                 # T_c(b_p)
    Qm, R = np.linalg.qr(V[use])
    coeffs = np.linalg.solve(R, Qm.T @ out[use].reshape(int(use.sum()), -1))   # Q x L Chebyshev coefficients
    out[flagged] = (V[flagged] @ coeffs).reshape((int(flagged.sum()),) + shape)
    return out


def rel_fro(a, b) -> float:
    """Relative Frobenius error ||a - b||_F / ||b||_F."""
    a, b = _f64(a), _f64(b)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))
