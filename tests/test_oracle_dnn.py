"""Pins of the oracle's DNN steps: finite-difference gradients, coded step = uncoded step."""

import numpy as np

from oracle import dnn
from oracle.code import GPCode
from oracle.locate import CORRECTED, NO_ERROR
from oracle.product import rel_fro


def _mlp(seed=0, widths=(12, 8, 8, 4), B=6):
    rng = np.random.default_rng(seed)
    Ws = [rng.standard_normal((widths[l + 1], widths[l])) * np.sqrt(2.0 / widths[l])
          for l in range(len(widths) - 1)]
    X = rng.standard_normal((widths[0], B))
    labels = rng.integers(0, widths[-1], size=B)
    return Ws, X, labels


def test_mlp_update_is_minus_lr_times_finite_difference_gradient():
    Ws, X, labels = _mlp()
    lr = 0.1
    new, info = dnn.mlp_step_uncoded(Ws, X, labels, lr)
    rng = np.random.default_rng(1)
    h = 1e-6
    for l in range(len(Ws)):
        for _ in range(6):
            i, j = rng.integers(0, Ws[l].shape[0]), rng.integers(0, Ws[l].shape[1])
            Wp = [w.copy() for w in Ws]
            Wm = [w.copy() for w in Ws]
            Wp[l][i, j] += h
            Wm[l][i, j] -= h
            g = (dnn.mlp_loss(Wp, X, labels) - dnn.mlp_loss(Wm, X, labels)) / (2 * h)
            assert np.isclose((new[l][i, j] - Ws[l][i, j]) / lr, -g, rtol=1e-5, atol=1e-8)


def test_backprop_recursion_matches_lemma():
    """delta^{l-1} = (W^l^T delta^l) o f'(s^{l-1}) with f'(s) = g(f(s))."""
    Ws, X, labels = _mlp(seed=2)
    _, info = dnn.mlp_step_uncoded(Ws, X, labels, 0.1)
    for l in range(len(Ws) - 1, 0, -1):
        want = (Ws[l].T @ info["Delta"][l]) * (info["S"][l - 1] > 0)
        assert np.allclose(info["Delta"][l - 1], want)


def test_autoencoder_update_matches_finite_differences():
    rng = np.random.default_rng(3)
    nv, nh, B = 10, 16, 7
    W1 = rng.standard_normal((nh, nv)) / np.sqrt(nv)
    W2 = rng.standard_normal((nv, nh)) / np.sqrt(nh)
    X = rng.uniform(0, 1, (nv, B)) * (rng.uniform(0, 1, (nv, B)) > 0.5)
    lr, rho, beta = 0.05, 0.05, 3.0
    n1, n2, loss = dnn.autoencoder_step_uncoded(W1, W2, X, lr, rho, beta)
    assert np.isclose(loss, dnn.autoencoder_loss(W1, W2, X, rho, beta))
    h = 1e-6
    for (W, new, which) in ((W1, n1, 0), (W2, n2, 1)):
        for _ in range(8):
            i, j = rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1])
            Wp, Wm = W.copy(), W.copy()
            Wp[i, j] += h
            Wm[i, j] -= h
            a = (Wp, W2) if which == 0 else (W1, Wp)
            b = (Wm, W2) if which == 0 else (W1, Wm)
            g = (dnn.autoencoder_loss(*a, X, rho, beta) - dnn.autoencoder_loss(*b, X, rho, beta)) / (2 * h)
            assert np.isclose((new[i, j] - W[i, j]) / lr, -g, rtol=1e-5, atol=1e-8)


def test_coded_mlp_step_equals_uncoded_step_with_and_without_errors():
    widths, B = (16, 12, 8, 4), 6
    Ws, X, labels = _mlp(seed=4, widths=widths, B=B)
    new, info = dnn.mlp_step_uncoded(Ws, X, labels, 0.01)
    for prob, seed in ((0.0, None), (0.15, 77)):
        layers = []
        for l, W in enumerate(Ws):
            code = GPCode(W.shape[0], W.shape[1], B, 2, 2, 1, 1, 10)
            layers.append(dnn.CodedLayer.from_weights(W, code, inject_mode="gauss", inject_prob=prob))
        out = dnn.mlp_step_coded(layers, X, labels, 0.01, step_seed=seed)
        assert out is not None
        for l in range(len(Ws)):
            assert rel_fro(out["S"][l], info["S"][l]) < 1e-9
            assert rel_fro(out["CT"][l], info["CT"][l]) < 1e-9
            W_dec, res = layers[l].audit()
            assert res.outcome == NO_ERROR and rel_fro(W_dec, new[l]) < 1e-10
        outcomes = [r.outcome for lay in layers for r in lay.log]
        if prob > 0:
            assert CORRECTED in outcomes          # the seed was chosen so that some node is hit
        else:
            assert set(outcomes) == {NO_ERROR}


def test_coded_autoencoder_steps_track_uncoded_training():
    rng = np.random.default_rng(5)
    nv, nh, B = 16, 32, 8
    W1 = rng.standard_normal((nh, nv)) / np.sqrt(nv)
    W2 = rng.standard_normal((nv, nh)) / np.sqrt(nh)
    X = rng.uniform(0, 1, (nv, B)) * (rng.uniform(0, 1, (nv, B)) > 0.5)
    enc = dnn.CodedLayer.from_weights(W1, GPCode(nh, nv, B, 2, 2, 1, 1, 10), inject_mode="gauss", inject_prob=0.1)
    dec = dnn.CodedLayer.from_weights(W2, GPCode(nv, nh, B, 2, 2, 1, 1, 10), inject_mode="gauss", inject_prob=0.1)
    U1, U2 = W1.copy(), W2.copy()
    losses = []
    for step in range(3):
        out = dnn.autoencoder_step_coded(enc, dec, X, 0.05, 0.05, 3.0, step_seed=1000 + 100 * step)
        assert out is not None
        U1, U2, loss = dnn.autoencoder_step_uncoded(U1, U2, X, 0.05, 0.05, 3.0)
        assert np.isclose(out["loss"], loss, rtol=1e-9)
        losses.append(loss)
    assert losses[-1] < losses[0]
    assert rel_fro(enc.audit()[0], U1) < 1e-9 and rel_fro(dec.audit()[0], U2) < 1e-9


def test_training_with_share_errors_and_regeneration_tracks_uncoded_training():
    """Errors left in the shares by the update stage surface at the next forward product, are
    located there and the shares regenerated (Section VI); the decoded weights keep following
    the uncoded SGD trajectory over several iterations."""
    widths, B = (16, 12, 8, 4), 6
    Ws, X, labels = _mlp(seed=6, widths=widths, B=B)
    layers = [dnn.CodedLayer.from_weights(W, GPCode(W.shape[0], W.shape[1], B, 2, 2, 1, 1, 10), inject_mode="gauss",
                                          inject_prob=0.08, regenerate=True, inject_shares=True) for W in Ws]
    U = [w.copy() for w in Ws]
    hits = 0
    for step in range(6):
        out = dnn.mlp_step_coded(layers, X, labels, 0.05, step_seed=5000 + 100 * step)
        assert out is not None
        U, info = dnn.mlp_step_uncoded(U, X, labels, 0.05)
        for l in range(len(Ws)):
            assert rel_fro(out["S"][l], info["S"][l]) < 1e-8
    for lay in layers:
        hits += sum(r.outcome == CORRECTED for r in lay.log)
    assert hits >= 3
    # one last forward pass repairs whatever the last update left behind, then the shares are clean
    for l, lay in enumerate(layers):
        lay.forward(info["X"][l] if l < len(info["X"]) else info["X"][-1], seed=None)
        W_dec, res = lay.audit()
        assert res.outcome == NO_ERROR and rel_fro(W_dec, U[l]) < 1e-8
