"""GPU parity of the coded training step (coded_layer_step and the element-wise kernels) against
the oracle's coded and uncoded FP64 steps, on reduced-size versions of the MLP and sparse
autoencoder workloads (same splits, node counts, error probability)."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import paper_1811_10751_b200 as g                      # noqa: E402
import workloads as wl                                 # noqa: E402
from oracle import dnn as odnn                         # noqa: E402
from oracle import product as op                       # noqa: E402
from oracle.code import GPCode                         # noqa: E402
from tests.gpu_pipeline import dev, host               # noqa: E402

REL_TOL = 1e-4


class GpuLayer:
    """Device state of one coded layer: plan, shares, workspace, results, outputs."""

    def __init__(self, W: np.ndarray, B: int, m: int, n: int, P: int, precision: int = g.GPD_PREC_AUTO):
        N1, N0 = W.shape
        self.N1, self.N0, self.B, self.P = N1, N0, B, P
        self.plan = g.gpd_plan((N1, N0, B), (m, n, 1, 1), P, precision=precision)
        self.np_dtype = np.float32 if self.plan.query(g.GPD_Q_ELEMENT_SIZE) == 4 else np.float64
        self.W_shares = self.plan.empty(g.GPD_Q_W_SHARE_ELEMS)
        g.gpd_encode_A(self.plan, dev(W), self.W_shares)
        self.ws = self.plan.workspace(step=True)
        self.res = g.new_results(3)
        f32 = dict(dtype=torch.float32, device="cuda")
        self.S = torch.full((N1, B), float("nan"), **f32)
        self.Xnext = torch.full((N1, B), float("nan"), **f32)
        self.CT = torch.full((B, N0), float("nan"), **f32)

    def step(self, phases, X=None, Delta=None, DeltaT=None, act=g.GPD_ACT_IDENTITY, eta=0.0, seed=0, prob=0.0):
        g.coded_layer_step(self.plan, phases, self.W_shares, X=X, Delta=Delta, DeltaT=DeltaT, activation=act,
                           eta=eta, inject_seed=seed, inject_prob=prob, inject_scale=1.0, S_out=self.S,
                           Xnext_out=self.Xnext, CT_out=self.CT, results=self.res, workspace=self.ws)

    def results(self):
        return g.read_results(self.res)

    def audit(self) -> np.ndarray:
        W = torch.empty((self.N1, self.N0), dtype=torch.float32, device="cuda")
        small = self.plan.workspace()
        r = g.new_results(1)
        g.gpd_locate_errors(self.plan, g.GPD_AUDIT, self.W_shares, r, small)
        g.gpd_decode(self.plan, g.GPD_AUDIT, self.W_shares, W, small, result=r)
        assert g.read_results(r)[0].outcome == g.GPD_NO_ERROR
        return host(W)


def _flags(r, P):
    return np.array(list(r.flagged)[:P], dtype=bool)


@pytest.mark.parametrize("prob,step_seed", [(0.0, 0), (0.05, 4321)])
def test_mlp_step_matches_oracle(prob, step_seed):
    _run_mlp_step(wl.scaled_down(wl.CONFIG_4_MLP, 16), prob, step_seed)   # 256-256-256-256-10, batch 16


def test_config4_full_size_step():
    """The MLP workload as stated: 4096-4096-4096-4096-10, batch 256, split 2 x 2, P = 10, one SGD step
    with every layer's forward product, backward product and update coded and node errors of
    probability 0.05 (the last layer's W has 5-row blocks: the small-block kernels)."""
    cfg = wl.CONFIG_4_MLP
    assert cfg.widths == (4096, 4096, 4096, 4096, 10) and cfg.B == 256 and cfg.P == 10
    _run_mlp_step(cfg, cfg.inject_prob, 4321)
    assert g.gpd_device_status() == 0


def _run_mlp_step(cfg, prob, step_seed):
    Ws, X1, labels = wl.mlp_inputs(cfg)
    L = len(Ws)
    # oracle: coded step (FP32 storage of worker outputs, same seeds) and uncoded FP64 step
    o_layers = []
    for W in Ws:
        code = GPCode(W.shape[0], W.shape[1], cfg.B, cfg.m, cfg.n, 1, 1, cfg.P)
        o_layers.append(odnn.CodedLayer.from_weights(W, code, out_dtype=np.float32, inject_mode="gauss",
                                                     inject_prob=prob))
    o_out = odnn.mlp_step_coded(o_layers, X1, labels, cfg.lr, step_seed=step_seed if prob > 0 else None)
    assert o_out is not None
    new_Ws, ref = odnn.mlp_step_uncoded(Ws, X1, labels, cfg.lr)

    layers = [GpuLayer(W, cfg.B, cfg.m, cfg.n, cfg.P) for W in Ws]
    assert all(l.np_dtype == np.float32 for l in layers)
    Xs = [dev(X1)]
    for l in range(L):
        act = g.GPD_ACT_RELU if l < L - 1 else g.GPD_ACT_IDENTITY
        layers[l].step(g.GPD_PHASE_FWD, X=Xs[l], act=act, seed=odnn.product_seed(step_seed, l, 0), prob=prob)
        Xs.append(layers[l].Xnext)
    C = Ws[-1].shape[0]
    Delta = torch.empty((C, cfg.B), dtype=torch.float32, device="cuda")
    DeltaT = torch.empty((cfg.B, C), dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    g.gpd_softmax_xent_delta(layers[-1].S, dev(labels.astype(np.int32)), Delta, DeltaT, loss)
    assert abs(float(loss.item()) - ref["loss"]) < 1e-4 * max(1.0, abs(ref["loss"]))
    deltas = [None] * L
    for l in range(L - 1, -1, -1):
        deltas[l] = Delta
        layers[l].step(g.GPD_PHASE_BWD | g.GPD_PHASE_UPD, X=Xs[l], Delta=Delta, DeltaT=DeltaT, eta=cfg.lr,
                       seed=odnn.product_seed(step_seed, l, 0), prob=prob)
        if l > 0:
            N = Ws[l].shape[1]
            Delta = torch.empty((N, cfg.B), dtype=torch.float32, device="cuda")
            DeltaT = torch.empty((cfg.B, N), dtype=torch.float32, device="cuda")
            g.gpd_backprop_hadamard(g.GPD_ACT_RELU, layers[l].CT, Xs[l], Delta, DeltaT)
    torch.cuda.synchronize()
    n_corrected = 0
    for l in range(L):
        rf, rb, _ = layers[l].results()
        of, ob = o_layers[l].log[0], o_layers[l].log[1]
        assert rf.outcome == of.outcome and np.array_equal(_flags(rf, cfg.P), of.flagged)
        assert rb.outcome == ob.outcome and np.array_equal(_flags(rb, cfg.P), ob.flagged)
        n_corrected += (rf.outcome == g.GPD_CORRECTED) + (rb.outcome == g.GPD_CORRECTED)
        assert op.rel_fro(host(layers[l].S), o_out["S"][l]) < REL_TOL
        assert op.rel_fro(host(layers[l].S), ref["S"][l]) < REL_TOL
        assert op.rel_fro(host(layers[l].CT), o_out["CT"][l]) < REL_TOL
        assert op.rel_fro(host(layers[l].CT), ref["CT"][l]) < REL_TOL
        assert op.rel_fro(host(deltas[l]), ref["Delta"][l]) < REL_TOL
        W_gpu = layers[l].audit()
        assert op.rel_fro(W_gpu, new_Ws[l]) < REL_TOL
        # the update itself (not only W) must be right: compare the weight change
        assert op.rel_fro(W_gpu.astype(np.float64) - Ws[l], new_Ws[l] - Ws[l].astype(np.float64)) < 5e-3
    if prob > 0:
        assert n_corrected >= 1                                # the seed was chosen to hit some node


def test_backward_failure_skips_the_update():
    """More erroneous nodes than P - Q_b - 1 in the backward product: decoding failure, no C^T
    written, shares untouched (the iteration would be redone from a checkpoint)."""
    W = np.random.default_rng(1).standard_normal((64, 64)).astype(np.float32)
    B, P = 8, 10
    layer = GpuLayer(W, B, 2, 2, P)
    before = layer.W_shares.clone()
    X = dev(np.random.default_rng(2).standard_normal((64, B)).astype(np.float32))
    Delta = dev(np.random.default_rng(3).standard_normal((64, B)).astype(np.float32))
    DeltaT = Delta.t().contiguous()
    layer.CT.fill_(5.0)
    layer.step(g.GPD_PHASE_BWD | g.GPD_PHASE_UPD, X=X, Delta=Delta, DeltaT=DeltaT, eta=0.1, seed=1, prob=0.9)
    torch.cuda.synchronize()
    _, rb, _ = layer.results()
    assert rb.outcome == g.GPD_DECODE_FAILURE
    assert bool((layer.CT == 5.0).all()) and torch.equal(layer.W_shares, before)
    # without errors the same call does update
    layer.step(g.GPD_PHASE_BWD | g.GPD_PHASE_UPD, X=X, Delta=Delta, DeltaT=DeltaT, eta=0.1)
    torch.cuda.synchronize()
    assert layer.results()[1].outcome == g.GPD_NO_ERROR and not torch.equal(layer.W_shares, before)


def test_sparse_autoencoder_steps_match_oracle():
    cfg = wl.scaled_down(wl.CONFIG_5_AUTOENCODER, 8)           # 128 <-> 1024, batch 128, P = 36, FP64 path
    W1, W2, X = wl.autoencoder_inputs(cfg)
    steps = 3
    enc_o = odnn.CodedLayer.from_weights(W1, GPCode(cfg.n_hidden, cfg.n_visible, cfg.B, cfg.m, cfg.n, 1, 1, cfg.P),
                                         inject_mode="gauss", inject_prob=cfg.inject_prob)
    dec_o = odnn.CodedLayer.from_weights(W2, GPCode(cfg.n_visible, cfg.n_hidden, cfg.B, cfg.m, cfg.n, 1, 1, cfg.P),
                                         inject_mode="gauss", inject_prob=cfg.inject_prob)
    enc, dec = GpuLayer(W1, cfg.B, cfg.m, cfg.n, cfg.P), GpuLayer(W2, cfg.B, cfg.m, cfg.n, cfg.P)
    assert enc.np_dtype == np.float64
    Xd = dev(X)
    U1, U2 = W1.astype(np.float64), W2.astype(np.float64)
    f32 = dict(dtype=torch.float32, device="cuda")
    D2, D2T = torch.empty((cfg.n_visible, cfg.B), **f32), torch.empty((cfg.B, cfg.n_visible), **f32)
    D1, D1T = torch.empty((cfg.n_hidden, cfg.B), **f32), torch.empty((cfg.B, cfg.n_hidden), **f32)
    mse, kl = torch.zeros(1, **f32), torch.zeros(1, **f32)
    for s in range(steps):
        seed = 9000 + 100 * s
        o = odnn.autoencoder_step_coded(enc_o, dec_o, X, cfg.lr, cfg.rho, cfg.beta, step_seed=seed)
        assert o is not None
        U1, U2, loss_ref = odnn.autoencoder_step_uncoded(U1, U2, X, cfg.lr, cfg.rho, cfg.beta)

        enc.step(g.GPD_PHASE_FWD, X=Xd, act=g.GPD_ACT_SIGMOID, seed=odnn.product_seed(seed, 0, 0), prob=cfg.inject_prob)
        dec.step(g.GPD_PHASE_FWD, X=enc.Xnext, seed=odnn.product_seed(seed, 1, 0), prob=cfg.inject_prob)
        g.gpd_sae_output_delta(dec.S, Xd, D2, D2T, mse)
        dec.step(g.GPD_PHASE_BWD, DeltaT=D2T, seed=odnn.product_seed(seed, 1, 0), prob=cfg.inject_prob)
        g.gpd_sae_hidden_delta(dec.CT, enc.Xnext, cfg.rho, cfg.beta, D1, D1T, kl)
        enc.step(g.GPD_PHASE_BWD | g.GPD_PHASE_UPD, X=Xd, Delta=D1, DeltaT=D1T, eta=cfg.lr,
                 seed=odnn.product_seed(seed, 0, 0), prob=cfg.inject_prob)
        dec.step(g.GPD_PHASE_UPD, X=enc.Xnext, Delta=D2, eta=cfg.lr)
        torch.cuda.synchronize()
        loss = float(mse.item() + kl.item())
        assert abs(loss - o["loss"]) < 1e-4 * abs(o["loss"]) and abs(loss - loss_ref) < 1e-4 * abs(loss_ref)
        assert op.rel_fro(host(enc.S), o["S1"]) < REL_TOL and op.rel_fro(host(dec.S), o["S2"]) < REL_TOL
        assert op.rel_fro(host(D1), o["Delta1"]) < REL_TOL and op.rel_fro(host(D2), o["Delta2"]) < REL_TOL
        assert op.rel_fro(host(enc.CT), o["C1T"]) < REL_TOL
        for lay, olay in ((enc, enc_o), (dec, dec_o)):         # outcome and flag vector of every product
            rf, rb, _ = lay.results()
            of, ob = olay.log[2 * s], olay.log[2 * s + 1]
            assert rf.outcome == of.outcome and np.array_equal(_flags(rf, cfg.P), of.flagged)
            assert rb.outcome == ob.outcome and np.array_equal(_flags(rb, cfg.P), ob.flagged)
    # flags of every product, in the order the oracle logged them
    assert len(enc_o.log) == 2 * steps and len(dec_o.log) == 2 * steps
    assert op.rel_fro(enc.audit(), U1) < REL_TOL and op.rel_fro(dec.audit(), U2) < REL_TOL
    assert op.rel_fro(enc.audit().astype(np.float64) - W1, U1 - W1) < 5e-3


@pytest.mark.parametrize("N1,N0,B,m,n,P,nodes", [
    (256, 256, 16, 2, 2, 10, (3, 8)),                      # FP32 storage, mn = 4
    (256, 128, 64, 4, 4, 36, (0, 5, 17, 30)),              # FP64 storage, mn = 16
])
def test_regenerate_shares_matches_oracle(N1, N0, B, m, n, P, nodes):
    W = (np.random.default_rng(31).standard_normal((N1, N0)) / np.sqrt(N0)).astype(np.float32)
    layer = GpuLayer(W, B, m, n, P)
    code = GPCode(N1, N0, B, m, n, 1, 1, P)
    clean = layer.W_shares.clone()
    mask = sum(1 << p for p in nodes)
    g.gpd_inject(layer.plan, g.GPD_AUDIT, layer.W_shares, 5, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=mask, scale=0.3)
    small, r = layer.plan.workspace(), g.new_results(1)
    g.gpd_locate_errors(layer.plan, g.GPD_AUDIT, layer.W_shares, r, small)
    res = g.read_results(r)[0]
    assert res.outcome == g.GPD_CORRECTED and list(np.flatnonzero(_flags(res, P))) == list(nodes)
    g.gpd_regenerate_shares(layer.plan, layer.W_shares, r, small)
    got = host(layer.W_shares).reshape(P, N1 // m, N0 // n).astype(np.float64)
    # oracle: its own encoding, the same nodes overwritten by anything, regenerated
    sh = op.encode_W(W, code)
    flagged = np.zeros(P, dtype=bool)
    flagged[list(nodes)] = True
    bad = sh.copy()
    bad[flagged] = 123.0
    want = op.regenerate_shares(bad, code, flagged)
    # a regenerated share must be as good as an encoded one (a few units of the storage rounding):
    # later products amplify any excess by up to 1e8 at thresholds near 30
    eps = 6e-8 if layer.np_dtype == np.float32 else 1.2e-16
    assert np.abs(got - want).max() <= 32 * eps * np.abs(want).max()
    assert np.abs(got - sh).max() <= 32 * eps * np.abs(sh).max()
    assert torch.equal(layer.W_shares.reshape(P, -1)[~torch.from_numpy(flagged).cuda()],
                       clean.reshape(P, -1)[~torch.from_numpy(flagged).cuda()])      # clean shares untouched
    # a clean audit regenerates nothing
    g.gpd_locate_errors(layer.plan, g.GPD_AUDIT, layer.W_shares, r, small)
    assert g.read_results(r)[0].outcome == g.GPD_NO_ERROR
    before = layer.W_shares.clone()
    g.gpd_regenerate_shares(layer.plan, layer.W_shares, r, small)
    assert torch.equal(layer.W_shares, before)


def test_training_with_share_errors_and_regeneration():
    """Several coded MLP iterations with soft errors in the products and in the updated shares;
    forward products locate the damaged nodes and their shares are regenerated (Section VI)."""
    cfg = wl.scaled_down(wl.CONFIG_4_MLP, 16)
    Ws, X1, labels = wl.mlp_inputs(cfg)
    L, prob, steps = len(Ws), 0.05, 4
    o_layers = [odnn.CodedLayer.from_weights(W, GPCode(W.shape[0], W.shape[1], cfg.B, cfg.m, cfg.n, 1, 1, cfg.P),
                                             out_dtype=np.float32, inject_mode="gauss", inject_prob=prob,
                                             regenerate=True, inject_shares=True) for W in Ws]
    layers = [GpuLayer(W, cfg.B, cfg.m, cfg.n, cfg.P) for W in Ws]
    U = [w.astype(np.float64) for w in Ws]
    labels_d = dev(labels.astype(np.int32))
    n_corrected = 0
    for it in range(steps):
        seed = 7000 + 100 * it
        o_out = odnn.mlp_step_coded(o_layers, X1, labels, cfg.lr, step_seed=seed)
        assert o_out is not None
        U, ref = odnn.mlp_step_uncoded(U, X1, labels, cfg.lr)
        Xs = [dev(X1)]
        for l in range(L):
            act = g.GPD_ACT_RELU if l < L - 1 else g.GPD_ACT_IDENTITY
            layers[l].step(g.GPD_PHASE_FWD | g.GPD_PHASE_REGEN, X=Xs[l], act=act, seed=odnn.product_seed(seed, l, 0),
                           prob=prob)
            Xs.append(layers[l].Xnext.clone())
        C = Ws[-1].shape[0]
        Delta = torch.empty((C, cfg.B), dtype=torch.float32, device="cuda")
        DeltaT = torch.empty((cfg.B, C), dtype=torch.float32, device="cuda")
        g.gpd_softmax_xent_delta(layers[-1].S, labels_d, Delta, DeltaT, None)
        for l in range(L - 1, -1, -1):
            layers[l].step(g.GPD_PHASE_BWD | g.GPD_PHASE_UPD | g.GPD_PHASE_INJECT_SHARES, X=Xs[l], Delta=Delta,
                           DeltaT=DeltaT, eta=cfg.lr, seed=odnn.product_seed(seed, l, 0), prob=prob)
            if l > 0:
                N = Ws[l].shape[1]
                Delta = torch.empty((N, cfg.B), dtype=torch.float32, device="cuda")
                DeltaT = torch.empty((cfg.B, N), dtype=torch.float32, device="cuda")
                g.gpd_backprop_hadamard(g.GPD_ACT_RELU, layers[l].CT, Xs[l], Delta, DeltaT)
        torch.cuda.synchronize()
        for l in range(L):
            rf, rb, _ = layers[l].results()
            of, ob = o_layers[l].log[2 * it], o_layers[l].log[2 * it + 1]
            assert rf.outcome == of.outcome and np.array_equal(_flags(rf, cfg.P), of.flagged), (it, l)
            assert rb.outcome == ob.outcome and np.array_equal(_flags(rb, cfg.P), ob.flagged), (it, l)
            n_corrected += (rf.outcome == g.GPD_CORRECTED) + (rb.outcome == g.GPD_CORRECTED)
            assert op.rel_fro(host(layers[l].S), ref["S"][l]) < REL_TOL
            assert op.rel_fro(host(layers[l].CT), ref["CT"][l]) < REL_TOL
    assert n_corrected >= 3
    # one more forward pass repairs what the last update left in the shares; then the audit is clean
    for l in range(L):
        layers[l].step(g.GPD_PHASE_FWD | g.GPD_PHASE_REGEN, X=dev(ref["X"][l].astype(np.float32)))
        torch.cuda.synchronize()
        assert op.rel_fro(layers[l].audit(), U[l]) < REL_TOL


@pytest.mark.parametrize("precision", [g.GPD_PREC_AUTO, g.GPD_PREC_FP64_SLICED_TRAIN])
def test_config5_full_size_two_steps(precision):
    """The sparse-autoencoder workload at full size (1024 <-> 8192, batch 1024, split 4 x 4, P = 36,
    thresholds 19 / 28 / 16), two coded SGD steps with Gaussian node errors: on the FP64 mma path the
    precision rule picks, and with every product on int8 digit planes (training mode)."""
    _run_autoencoder(wl.CONFIG_5_AUTOENCODER, 2, precision)


def test_config5_ten_steps_half_size():
    """All ten SGD steps of the workload, at half the width and batch (512 <-> 4096, batch 512; same
    split, node count, thresholds and error probability): the oracle's ten full-size steps take minutes."""
    cfg = wl.scaled_down(wl.CONFIG_5_AUTOENCODER, 2)
    assert cfg.steps == 10 and cfg.P == 36
    _run_autoencoder(cfg, cfg.steps, g.GPD_PREC_FP64_SLICED_TRAIN)


def _run_autoencoder(cfg, n_steps, precision):
    W1, W2, X = wl.autoencoder_inputs(cfg)
    enc_o = odnn.CodedLayer.from_weights(W1, GPCode(cfg.n_hidden, cfg.n_visible, cfg.B, cfg.m, cfg.n, 1, 1, cfg.P),
                                         inject_mode="gauss", inject_prob=cfg.inject_prob)
    dec_o = odnn.CodedLayer.from_weights(W2, GPCode(cfg.n_visible, cfg.n_hidden, cfg.B, cfg.m, cfg.n, 1, 1, cfg.P),
                                         inject_mode="gauss", inject_prob=cfg.inject_prob)
    enc = GpuLayer(W1, cfg.B, cfg.m, cfg.n, cfg.P, precision)
    dec = GpuLayer(W2, cfg.B, cfg.m, cfg.n, cfg.P, precision)
    assert enc.np_dtype == np.float64
    Xd = dev(X)
    U1, U2 = W1.astype(np.float64), W2.astype(np.float64)
    f32 = dict(dtype=torch.float32, device="cuda")
    D2, D2T = torch.empty((cfg.n_visible, cfg.B), **f32), torch.empty((cfg.B, cfg.n_visible), **f32)
    D1, D1T = torch.empty((cfg.n_hidden, cfg.B), **f32), torch.empty((cfg.B, cfg.n_hidden), **f32)
    mse, kl = torch.zeros(1, **f32), torch.zeros(1, **f32)
    n_corrected = 0
    for s in range(n_steps):
        seed = 8800 + 100 * s
        o = odnn.autoencoder_step_coded(enc_o, dec_o, X, cfg.lr, cfg.rho, cfg.beta, step_seed=seed)
        assert o is not None
        U1, U2, loss_ref = odnn.autoencoder_step_uncoded(U1, U2, X, cfg.lr, cfg.rho, cfg.beta)
        enc.step(g.GPD_PHASE_FWD, X=Xd, act=g.GPD_ACT_SIGMOID, seed=odnn.product_seed(seed, 0, 0), prob=cfg.inject_prob)
        dec.step(g.GPD_PHASE_FWD, X=enc.Xnext, seed=odnn.product_seed(seed, 1, 0), prob=cfg.inject_prob)
        g.gpd_sae_output_delta(dec.S, Xd, D2, D2T, mse)
        dec.step(g.GPD_PHASE_BWD, DeltaT=D2T, seed=odnn.product_seed(seed, 1, 0), prob=cfg.inject_prob)
        g.gpd_sae_hidden_delta(dec.CT, enc.Xnext, cfg.rho, cfg.beta, D1, D1T, kl)
        enc.step(g.GPD_PHASE_BWD | g.GPD_PHASE_UPD, X=Xd, Delta=D1, DeltaT=D1T, eta=cfg.lr,
                 seed=odnn.product_seed(seed, 0, 0), prob=cfg.inject_prob)
        dec.step(g.GPD_PHASE_UPD, X=enc.Xnext, Delta=D2, eta=cfg.lr)
        torch.cuda.synchronize()
        loss = float(mse.item() + kl.item())
        assert abs(loss - loss_ref) < 1e-4 * abs(loss_ref)
        for lay, olay in ((enc, enc_o), (dec, dec_o)):
            rf, rb, _ = lay.results()
            of, ob = olay.log[2 * s], olay.log[2 * s + 1]
            assert rf.outcome == of.outcome and np.array_equal(_flags(rf, cfg.P), of.flagged)
            assert rb.outcome == ob.outcome and np.array_equal(_flags(rb, cfg.P), ob.flagged)
            n_corrected += (rf.outcome == g.GPD_CORRECTED) + (rb.outcome == g.GPD_CORRECTED)
        assert op.rel_fro(host(enc.S), o["S1"]) < REL_TOL and op.rel_fro(host(dec.S), o["S2"]) < REL_TOL
        assert op.rel_fro(host(D1), o["Delta1"]) < REL_TOL and op.rel_fro(host(D2), o["Delta2"]) < REL_TOL
        assert op.rel_fro(host(enc.CT), o["C1T"]) < REL_TOL
    assert n_corrected >= 1
    assert op.rel_fro(enc.audit(), U1) < REL_TOL and op.rel_fro(dec.audit(), U2) < REL_TOL
    assert g.gpd_device_status() == 0
