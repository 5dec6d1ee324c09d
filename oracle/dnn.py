"""Uncoded FP64 SGD steps and the coded layer step (test oracle; numpy).

Uncoded steps follow Section II-B and the DNN-background appendix: feedforward
S = W X, X_next = f(S); last-layer error; backpropagation C^T = Delta^T W,
Delta_prev^T = C^T o g(X^T); update W <- (1 - eta*lam) W + eta Delta X^T.
The backpropagated error is the *negative* gradient of the mini-batch loss with
respect to S (delta = -d eps^2 / d s), so updates add.

The coded step (Sections VI and VIII) keeps W~_p encoded: encode X (or Delta^T),
multiply at every node, locate erroneous nodes, interpolate the wanted
coefficients; the update is applied to the shares directly (Eq. 10).

Readings where the paper is silent: softmax cross-entropy's last-layer error is
(Y_onehot - softmax(S)) / B;  ReLU's g(x) = 1[x > 0];  the sparse-autoencoder loss
is  E = (1/B) sum_b ||S2_b - x_b||^2 + beta * sum_i KL(rho || rho_hat_i), which gives
Delta2 = (2/B)(X - S2) and Delta1 = (C2 - (beta/B) Q(rho_hat) 1^T) o Y1 o (1 - Y1).
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np

from . import inject as inj
from .code import GPCode, FWD, BWD, AUDIT
from .locate import LocateResult, locate_subspace, tolerances_for, DECODE_FAILURE
from .product import (decode, encode_DeltaT, encode_update_operands, encode_W, encode_X,
                      regenerate_shares, update_shares, worker_products)


# ------------------------------------------------------------------------------------------
# element-wise pieces (steps C1, C2 and the last-layer transition)
# ------------------------------------------------------------------------------------------
def relu(S):
    return np.maximum(S, 0.0)


def relu_g(X):
    """g with g(f(u)) = f'(u) for f = ReLU, applied to the layer's *input* X = f(S_prev)."""
    return (X > 0.0).astype(np.float64)


def sigmoid(S):
    return 1.0 / (1.0 + np.exp(-S))


def softmax_columns(S):
    E = np.exp(S - S.max(axis=0, keepdims=True))
    return E / E.sum(axis=0, keepdims=True)


def softmax_ce_loss(S, labels) -> float:
    Pm = softmax_columns(S)
    B = S.shape[1]
    return float(-np.log(Pm[labels, np.arange(B)]).mean())


def softmax_ce_delta(S, labels):
    """Negative gradient of the mean cross-entropy with respect to S (classes x B)."""
    B = S.shape[1]
    Y = np.zeros_like(S)
    Y[labels, np.arange(B)] = 1.0
    return (Y - softmax_columns(S)) / B


# ------------------------------------------------------------------------------------------
# uncoded MLP step
# ------------------------------------------------------------------------------------------
def mlp_loss(Ws: Sequence[np.ndarray], X1, labels) -> float:
    X = np.asarray(X1, dtype=np.float64)
    for l, W in enumerate(Ws):
        S = np.asarray(W, dtype=np.float64) @ X
        X = relu(S) if l < len(Ws) - 1 else S
    return softmax_ce_loss(X, labels)


def mlp_step_uncoded(Ws: Sequence[np.ndarray], X1, labels, lr: float):
    """One SGD step.  Returns (new weights, dict of intermediates)."""
    Ws = [np.asarray(W, dtype=np.float64) for W in Ws]
    L = len(Ws)
    Xs, Ss = [np.asarray(X1, dtype=np.float64)], []
    for l in range(L):
        S = Ws[l] @ Xs[l]
        Ss.append(S)
        if l < L - 1:
            Xs.append(relu(S))
    Delta = softmax_ce_delta(Ss[-1], labels)                 # N_L x B
    Deltas = [None] * L
    CTs = [None] * L
    for l in range(L - 1, -1, -1):
        Deltas[l] = Delta
        CT = Delta.T @ Ws[l]                                 # B x N_{l-1}
        CTs[l] = CT
        if l > 0:
            Delta = (CT * relu_g(Xs[l]).T).T
    new_Ws = [Ws[l] + lr * (Deltas[l] @ Xs[l].T) for l in range(L)]
    return new_Ws, {"X": Xs, "S": Ss, "Delta": Deltas, "CT": CTs,
                    "loss": softmax_ce_loss(Ss[-1], labels)}


# ------------------------------------------------------------------------------------------
# uncoded sparse-autoencoder step (Section IX and its appendix)
# ------------------------------------------------------------------------------------------
RHO_CLAMP = 1e-7


def kl_q(rho_hat, rho: float):
    """Q(rho_hat) = -rho/rho_hat + (1-rho)/(1-rho_hat)."""
    return -rho / rho_hat + (1.0 - rho) / (1.0 - rho_hat)


def autoencoder_loss(W1, W2, X, rho: float, beta: float) -> float:
    W1, W2, X = (np.asarray(a, dtype=np.float64) for a in (W1, W2, X))
    B = X.shape[1]
    Y1 = sigmoid(W1 @ X)
    S2 = W2 @ Y1
    rho_hat = np.clip(Y1.mean(axis=1), RHO_CLAMP, 1.0 - RHO_CLAMP)
    kl = rho * np.log(rho / rho_hat) + (1.0 - rho) * np.log((1.0 - rho) / (1.0 - rho_hat))
    return float(((S2 - X) ** 2).sum() / B + beta * kl.sum())


def autoencoder_deltas(S1, S2, C2T_fn, X, rho: float, beta: float):
    """Delta2 and, given a way to obtain C2^T = Delta2^T W2, Delta1."""
    B = X.shape[1]
    Y1 = sigmoid(S1)
    Delta2 = (2.0 / B) * (X - S2)
    C2T = C2T_fn(Delta2)                                     # B x N_hidden
    rho_hat = np.clip(Y1.mean(axis=1), RHO_CLAMP, 1.0 - RHO_CLAMP)
    Qv = kl_q(rho_hat, rho)
    Delta1 = (C2T.T - (beta / B) * Qv[:, None]) * Y1 * (1.0 - Y1)
    return Delta1, Delta2, Y1


def autoencoder_step_uncoded(W1, W2, X, lr: float, rho: float, beta: float):
    W1, W2, X = (np.asarray(a, dtype=np.float64) for a in (W1, W2, X))
    S1 = W1 @ X
    Y1 = sigmoid(S1)
    S2 = W2 @ Y1
    Delta1, Delta2, _ = autoencoder_deltas(S1, S2, lambda D2: D2.T @ W2, X, rho, beta)
    return W1 + lr * (Delta1 @ X.T), W2 + lr * (Delta2 @ Y1.T), autoencoder_loss(W1, W2, X, rho, beta)


# ------------------------------------------------------------------------------------------
# coded layer
# ------------------------------------------------------------------------------------------
@dataclass
class CodedLayer:
    """One layer whose weight matrix stays encoded as P shares W~_p."""

    code: GPCode
    W_shares: np.ndarray                 # [P][N1/m][N0/n], FP64
    out_dtype: type = np.float64         # storage type of worker outputs (decides tolerances)
    inject_mode: str = "none"            # "none" | "gauss" | "additive"
    inject_prob: float = 0.0
    inject_scale: float = 1.0
    regenerate: bool = False             # after a forward product, regenerate the shares of flagged nodes
    inject_shares: bool = False          # the update stage leaves Gaussian node errors in the shares
    log: List[LocateResult] = field(default_factory=list)

    @classmethod
    def from_weights(cls, W, code: GPCode, **kw) -> "CodedLayer":
        return cls(code=code, W_shares=encode_W(W, code), **kw)

    def _finish(self, outputs: np.ndarray, which: int, seed: Optional[int], scale: float):
        Z = outputs.astype(self.out_dtype)
        if seed is not None and self.inject_mode != "none":
            fn = inj.inject_gauss if self.inject_mode == "gauss" else inj.inject_additive
            fn(Z, seed, scale, prob=self.inject_prob)
        res = locate_subspace(Z, self.code.points, self.code.Q(which), tolerances_for(self.out_dtype))
        self.log.append(res)
        if res.outcome == DECODE_FAILURE:
            return None, res
        return decode(Z, self.code, which, use=~res.flagged), res

    def forward(self, X, seed: Optional[int] = None, scale: float = 1.0):
        """S = W X through encode -> P products -> locate -> decode."""
        Z = worker_products(self.W_shares, encode_X(X, self.code))
        S, res = self._finish(Z, FWD, seed, scale)
        if self.regenerate and S is not None and res.flagged.any():
            self.W_shares = regenerate_shares(self.W_shares, self.code, res.flagged)
        return S, res

    def backward(self, DeltaT, seed: Optional[int] = None, scale: float = 1.0):
        """C^T = Delta^T W through the same four stages."""
        Z = worker_products(encode_DeltaT(DeltaT, self.code), self.W_shares)
        return self._finish(Z, BWD, seed, scale)

    def update(self, Delta, X, eta: float, lam: float = 0.0, seed: Optional[int] = None, scale: float = 1.0):
        Dh, Xh = encode_update_operands(Delta, X, self.code)
        self.W_shares = update_shares(self.W_shares, Dh, Xh, eta, lam)
        if self.inject_shares and seed is not None and self.inject_prob > 0:
            inj.inject_gauss(self.W_shares, seed, scale, prob=self.inject_prob)

    def audit(self, seed: Optional[int] = None, scale: float = 1.0):
        """Decode W itself from the shares (each share is a degree mn-1 polynomial evaluation)."""
        return self._finish(self.W_shares.copy(), AUDIT, seed, scale)


def rms(a) -> float:
    a = np.asarray(a, dtype=np.float64)
    return float(np.sqrt(np.mean(a * a))) if a.size else 0.0


# ------------------------------------------------------------------------------------------
# coded training steps (composition of CodedLayer calls; one seed per product)
# ------------------------------------------------------------------------------------------
def product_seed(step_seed: int, layer: int, stage: int) -> int:
    """Seed of the injection after product `stage` (0 forward, 1 backward, 2 update) of `layer`."""
    return step_seed + 16 * layer + stage


def mlp_step_coded(layers: Sequence[CodedLayer], X1, labels, lr: float,
                   step_seed: Optional[int] = None):
    """One coded SGD step of a ReLU MLP with softmax cross-entropy.

    Returns a dict with the decoded S, C^T per layer, or None as soon as a product
    declares a decoding failure (the caller would restore a checkpoint)."""
    L = len(layers)
    sd = (lambda l, s: None) if step_seed is None else (lambda l, s: product_seed(step_seed, l, s))
    Xs, Ss = [np.asarray(X1, dtype=np.float64)], []
    for l in range(L):
        S, res = layers[l].forward(Xs[l], seed=sd(l, 0))
        if S is None:
            return None
        Ss.append(S)
        if l < L - 1:
            Xs.append(relu(S))
    Delta = softmax_ce_delta(Ss[-1], labels)
    Deltas, CTs = [None] * L, [None] * L
    for l in range(L - 1, -1, -1):
        Deltas[l] = Delta
        CT, res = layers[l].backward(Delta.T, seed=sd(l, 1))
        if CT is None:
            return None
        CTs[l] = CT
        if l > 0:
            Delta = (CT * relu_g(Xs[l]).T).T
    for l in range(L):
        layers[l].update(Deltas[l], Xs[l], lr, seed=sd(l, 2))
    return {"X": Xs, "S": Ss, "Delta": Deltas, "CT": CTs, "loss": softmax_ce_loss(Ss[-1], labels)}


def autoencoder_step_coded(enc: CodedLayer, dec: CodedLayer, X, lr: float, rho: float, beta: float,
                           step_seed: Optional[int] = None):
    """One coded SGD step of the sparse autoencoder; None on a decoding failure."""
    sd = (lambda l, s: None) if step_seed is None else (lambda l, s: product_seed(step_seed, l, s))
    X = np.asarray(X, dtype=np.float64)
    S1, r = enc.forward(X, seed=sd(0, 0))
    if S1 is None:
        return None
    Y1 = sigmoid(S1)
    S2, r = dec.forward(Y1, seed=sd(1, 0))
    if S2 is None:
        return None
    failed = []

    def c2t(D2):
        CT, res = dec.backward(D2.T, seed=sd(1, 1))
        if CT is None:
            failed.append(res)
            return np.zeros((X.shape[1], enc.code.N1))
        return CT

    Delta1, Delta2, _ = autoencoder_deltas(S1, S2, c2t, X, rho, beta)
    if failed:
        return None
    C1T, r = enc.backward(Delta1.T, seed=sd(0, 1))       # computed although unused (first layer)
    if C1T is None:
        return None
    B = X.shape[1]
    rho_hat = np.clip(Y1.mean(axis=1), RHO_CLAMP, 1.0 - RHO_CLAMP)
    kl = rho * np.log(rho / rho_hat) + (1.0 - rho) * np.log((1.0 - rho) / (1.0 - rho_hat))
    loss = float(((S2 - X) ** 2).sum() / B + beta * kl.sum())
    enc.update(Delta1, X, lr, seed=sd(0, 2))
    dec.update(Delta2, Y1, lr, seed=sd(1, 2))
    return {"S1": S1, "S2": S2, "Delta1": Delta1, "Delta2": Delta2, "C1T": C1T, "loss": loss}
