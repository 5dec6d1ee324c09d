"""GPU parity of the integer-slice product paths (GPD_PREC_FP64_SLICED, GPD_PREC_FP64_SLICED40,
GPD_PREC_FP64_SLICED_TRAIN) against the FP64 oracle.

The shares are stored as S = 6 (or 5) signed 8-bit digits per value under one power-of-two scale 2^e
per operand row.  For a column of X~_p, 2^e lies in (2.03, 4.07] times the column's largest magnitude;
for a row of W~_p it lies in the same range times the bound sum_b |coef_pb| max_c |W_b[r][c]| of the
row's magnitudes (W_b the blocks the share combines).
Digit-plane products are exact, so a worker output differs from the exact product of the FP64 shares
only by (i) the digits cut below 2^-(8S+1) of each scale and (ii) the plane pairs of weight below
256^-(S+1) that are not formed (S - 1 of them at the largest dropped weight, |digit| <= 128): per
term of the contraction at most 2^-(8S+1) + (S - 1) * 1.004 * 2^14 * 256^-(S+2) of 2^ea 2^eb, which is
6.5e-15 for S = 6 and 1.4e-12 for S = 5 (reached only with every digit at its largest value).  The
tests allow 4 sqrt(K) times that (signs of the per-term errors are independent); a single missing
plane pair of the kept set, 256 times heavier than the heaviest dropped one, exceeds it several
times over.
"""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import paper_1811_10751_b200 as g                        # noqa: E402
from oracle import product as op                         # noqa: E402
from oracle.code import GPCode, FWD, BWD                 # noqa: E402
from oracle.locate import NO_ERROR, CORRECTED, locate_subspace, tolerances_for   # noqa: E402
from oracle import inject as oinj                        # noqa: E402
from tests.gpu_pipeline import CodedProduct, dev, host   # noqa: E402

PER_TERM = {6: 6.5e-15, 5: 1.4e-12}
PRECISIONS = {6: g.GPD_PREC_FP64_SLICED, 5: g.GPD_PREC_FP64_SLICED40}
SCALE_OVER_MAX = 4.07


def _inputs(N1, N0, B, seed, w_scale=1.0, x_scale=1.0):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N1, N0)) / np.sqrt(N0) * w_scale).astype(np.float32)
    X = (rng.standard_normal((N0, B)) * x_scale).astype(np.float32)
    return W, X


def _row_bound(W, code):
    """sum_b |coef_pb| max_c |W_b[r][c]| for every node p and share row r: [P][M]."""
    M, K = code.N1 // code.m, code.N0 // code.n
    blkmax = np.abs(W.astype(np.float64)).reshape(code.m, M, code.n, K).max(axis=3)      # [m][M][n]
    coef = np.abs(code.points)[:, None, None] ** code.exp_W()[None, :, :]                 # [P][m][n]
    return np.einsum("pij,irj->pr", coef, blkmax)


def _output_tolerance(W, code, Wsh, Xsh, S=6):
    """Per-entry bound [P][M][N] from the inputs and the oracle's FP64 shares (see the module docstring)."""
    K = Wsh.shape[2]
    row = SCALE_OVER_MAX * _row_bound(W, code)             # [P][M]  >= 2^ea
    assert (row >= SCALE_OVER_MAX * np.abs(Wsh).max(axis=2) * (1 - 1e-12)).all()
    col = SCALE_OVER_MAX * np.abs(Xsh).max(axis=1)         # [P][N]  >= 2^eb
    return 4.0 * np.sqrt(K) * PER_TERM[S] * row[:, :, None] * col[:, None, :]


def _sliced_products(code, W, X, S=6):
    cp = CodedProduct(code, precision=PRECISIONS[S])
    assert cp.plan.query(g.GPD_Q_PRECISION) == PRECISIONS[S] and cp.np_dtype == np.float64
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    assert g.gpd_device_status() == 0
    return cp, Z


@pytest.mark.parametrize("N1,N0,B,m,n,d1,P", [
    (256, 256, 128, 2, 4, 2, 25),       # whole tiles
    (400, 320, 144, 2, 4, 2, 25),       # ragged rows (200 = 128 + 72) and columns (72 = 64 + 8), K = 80
    (384, 96, 66, 3, 2, 2, 20),         # 6 blocks per share of W, K = 48 (one partly filled k-block), odd column count
    (130, 16, 4, 1, 1, 1, 4),           # K = 16, single block, two columns
    (1024, 2048, 128, 2, 2, 1, 9),      # K = 1024: sixteen k-blocks, ring wraps five times
    (512, 768, 96, 4, 4, 1, 40),        # 16 blocks per share of W, 40 nodes, threshold 19
    (256, 256, 96, 2, 4, 3, 30),        # 12 blocks per share of X, threshold 27
    (128, 16384, 32, 2, 2, 1, 8),       # K = 8192: share rows too long for the encoder's shared-memory staging
])
@pytest.mark.parametrize("S", [6, 5])
def test_sliced_worker_products_match_oracle(N1, N0, B, m, n, d1, P, S):
    W, X = _inputs(N1, N0, B, seed=N1 + N0 + B)
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    cp, Z = _sliced_products(code, W, X, S)
    Wsh, Xsh = op.encode_W(W, code), op.encode_X(X, code)
    Zo = op.worker_products(Wsh, Xsh)
    got = cp.outputs_as_array(g.GPD_FWD, Z)
    assert np.isfinite(got).all()
    tol = _output_tolerance(W, code, Wsh, Xsh, S)
    assert (np.abs(got - Zo) <= tol).all(), float((np.abs(got - Zo) / tol).max())
    # and the bound is far below what FP32 shares could give: relative to the output scale
    assert np.abs(got - Zo).max() < (1e-10 if S == 6 else 2e-8) * np.sqrt(np.mean(Zo ** 2))


@pytest.mark.parametrize("N1,N0,B,m,n,d1,P,S", [(256, 512, 128, 2, 4, 2, 25, 6), (192, 96, 64, 3, 2, 2, 20, 5),
                                                (256, 256, 64, 2, 2, 1, 8, 6)])
def test_sliced_products_with_the_library_points(N1, N0, B, m, n, d1, P, S):
    """The library's own evaluation points (Chebyshev, mirrored exactly: b_{P-1-p} = -b_p, 0 in the
    middle for odd P) instead of the oracle's; the oracle is given the same points."""
    plan0 = g.gpd_plan((N1, N0, B), (m, n, d1, 1), P)
    pts = plan0.table(g.GPD_TABLE_POINTS)
    plan0.destroy()
    assert np.array_equal(pts, -pts[::-1]) and np.all(np.diff(pts) < 0)
    W, X = _inputs(N1, N0, B, seed=N1 + P)
    code = GPCode(N1, N0, B, m, n, d1, 1, P, points=pts)
    cp, Z = _sliced_products(code, W, X, S)
    Wsh, Xsh = op.encode_W(W, code), op.encode_X(X, code)
    got = cp.outputs_as_array(g.GPD_FWD, Z)
    tol = _output_tolerance(W, code, Wsh, Xsh, S)
    assert (np.abs(got - op.worker_products(Wsh, Xsh)) <= tol).all()
    r = cp.locate(g.GPD_FWD, Z)
    assert r.outcome == NO_ERROR
    assert op.rel_fro(cp.decode(g.GPD_FWD, Z), op.ref_forward(W, X)) < 1e-4


def test_sliced_products_alternate_substitution_with_the_library_points():
    """The substitution v = u^m, w = u^(mn) gives W's block (i, j) the exponent i + m j; with mirrored
    points the encoder evaluates the share polynomial of nodes p and P-1-p from shared even and odd halves
    and has to pick the blocks in the order of their exponents."""
    from oracle.code import SUBST_V_UM
    N1, N0, B, m, n, d1, P = 192, 256, 64, 3, 2, 2, 21
    plan0 = g.gpd_plan((N1, N0, B), (m, n, d1, 1), P)
    pts = plan0.table(g.GPD_TABLE_POINTS)
    plan0.destroy()
    W, X = _inputs(N1, N0, B, seed=77)
    code = GPCode(N1, N0, B, m, n, d1, 1, P, points=pts, subst=SUBST_V_UM)
    assert P >= code.Q_f
    cp, Z = _sliced_products(code, W, X)
    Wsh, Xsh = op.encode_W(W, code), op.encode_X(X, code)
    got = cp.outputs_as_array(g.GPD_FWD, Z)
    assert (np.abs(got - op.worker_products(Wsh, Xsh)) <= _output_tolerance(W, code, Wsh, Xsh)).all()
    assert op.rel_fro(cp.decode(g.GPD_FWD, Z), op.ref_forward(W, X)) < 1e-4


def test_sliced_scales_zero_rows_and_tiny_values():
    """Row / column scales: rows of zeros, columns of zeros and operands 1e-30 and 1e+20 times the
    usual size decode to the same relative accuracy (the digits carry no absolute scale)."""
    N1, N0, B, m, n, d1, P = 256, 128, 96, 2, 2, 2, 12
    W, X = _inputs(N1, N0, B, seed=5, w_scale=1e-30, x_scale=1e20)
    W[7, :] = 0.0                       # zero row in block 0
    W[128 + 7, :] = 0.0                 # and the same row of block 1: share row 7 is zero on every node
    X[:, 5] = 0.0
    X[:, 48 + 5] = 0.0                  # share column 5 is zero on every node
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    cp, Z = _sliced_products(code, W, X)
    Wsh, Xsh = op.encode_W(W, code), op.encode_X(X, code)
    Zo = op.worker_products(Wsh, Xsh)
    got = cp.outputs_as_array(g.GPD_FWD, Z)
    assert (got[:, 7, :] == 0.0).all() and (got[:, :, 5] == 0.0).all()
    assert (np.abs(got - Zo) <= _output_tolerance(W, code, Wsh, Xsh)).all()
    r = cp.locate(g.GPD_FWD, Z)
    assert r.outcome == NO_ERROR
    S = cp.decode(g.GPD_FWD, Z)
    assert op.rel_fro(S, op.ref_forward(W, X)) < 1e-4


@pytest.mark.parametrize("S", [6, 5])
def test_sliced_pipeline_locates_and_decodes_like_the_oracle(S):
    N1, N0, B, m, n, d1, P = 512, 512, 128, 2, 4, 2, 25
    W, X = _inputs(N1, N0, B, seed=11)
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    cp, Z = _sliced_products(code, W, X, S)
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    scale = float(np.sqrt(np.mean(Zo ** 2)))
    ref = op.ref_forward(W, X)
    seen = set()
    for seed in range(300, 306):
        Zg = Z.clone()
        g.gpd_inject(cp.plan, g.GPD_FWD, Zg, seed, g.GPD_INJECT_ADDITIVE, prob=0.1, scale=scale)
        Zr = Zo.copy()
        sel = oinj.inject_additive(Zr, seed, scale, prob=0.1)
        ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
        r = cp.locate(g.GPD_FWD, Zg)
        assert r.outcome == ro.outcome and np.array_equal(cp.flags(r), ro.flagged)
        seen.add(r.outcome)
        if r.outcome in (NO_ERROR, CORRECTED):
            assert np.array_equal(ro.flagged, sel)
            S = cp.decode(g.GPD_FWD, Zg)
            assert op.rel_fro(S, ref) < 1e-4
            assert op.rel_fro(S, op.decode(Zr, code, FWD, use=~ro.flagged)) < 1e-4
    assert CORRECTED in seen


def test_sliced_layer_step_forward_only():
    N1, N0, B, m, n, d1, P = 256, 256, 64, 2, 2, 1, 9
    W, X = _inputs(N1, N0, B, seed=21)
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    plan = g.gpd_plan((N1, N0, B), (m, n, d1, 1), P, points=code.points, precision=g.GPD_PREC_FP64_SLICED)
    Wsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS)
    g.gpd_encode_A(plan, dev(W), Wsh)
    S = torch.full((N1, B), float("nan"), dtype=torch.float32, device="cuda")
    A = torch.full((N1, B), float("nan"), dtype=torch.float32, device="cuda")
    res, ws = g.new_results(2), plan.workspace(step=True)
    g.coded_layer_step(plan, g.GPD_PHASE_FWD, Wsh, X=dev(X), activation=g.GPD_ACT_RELU, inject_seed=70,
                       inject_prob=0.2, inject_scale=1.0, S_out=S, Xnext_out=A, results=res, workspace=ws)
    r = g.read_results(res)[0]
    Zr = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    sel = oinj.inject_gauss(Zr, 70, 1.0, prob=0.2)
    ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
    assert r.outcome == ro.outcome and np.array_equal(np.array(list(r.flagged)[:P], dtype=bool), ro.flagged)
    assert sel.any() and ro.outcome == CORRECTED
    ref = op.ref_forward(W, X)
    assert op.rel_fro(host(S), ref) < 1e-4
    assert op.rel_fro(host(A), np.maximum(ref, 0.0)) < 1e-4
    # every other phase needs shares this storage cannot serve
    for phases in (g.GPD_PHASE_FWD | g.GPD_PHASE_REGEN, g.GPD_PHASE_BWD, g.GPD_PHASE_UPD,
                   g.GPD_PHASE_FWD | g.GPD_PHASE_BWD | g.GPD_PHASE_UPD):
        with pytest.raises(g.GpdError) as ei:
            g.coded_layer_step(plan, phases, Wsh, X=dev(X), Delta=dev(np.zeros((N1, B), np.float32)),
                               DeltaT=dev(np.zeros((B, N1), np.float32)), S_out=S, Xnext_out=A,
                               CT_out=torch.empty((B, N0), dtype=torch.float32, device="cuda"), results=res, workspace=ws)
        assert ei.value.status == g.GPD_ERR_UNSUPPORTED


def test_sliced_refuses_calls_on_other_shares():
    N1, N0, B, m, n, d1, P = 128, 128, 32, 2, 2, 1, 9
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    cp = CodedProduct(code, precision=g.GPD_PREC_FP64_SLICED)
    W, X = _inputs(N1, N0, B, seed=3)
    cp.encode_W(W)
    for operand, M in ((g.GPD_OPERAND_DELTAT_BWD, np.zeros((B, N1), np.float32)),
                       (g.GPD_OPERAND_DELTA_UPD, np.zeros((N1, B), np.float32)),
                       (g.GPD_OPERAND_X_UPD, X)):
        with pytest.raises(g.GpdError) as ei:
            cp.encode(operand, M)
        assert ei.value.status == g.GPD_ERR_UNSUPPORTED
    Xs = cp.encode(g.GPD_OPERAND_X_FWD, X)
    # a source matrix that does not start on a 16-byte boundary is refused, not read with vector loads
    skew = torch.empty(N1 * N0 + 1, dtype=torch.float32, device="cuda")[1:].view(N1, N0)
    with pytest.raises(g.GpdError) as ei:
        g.gpd_encode_A(cp.plan, skew, cp.W_shares)
    assert ei.value.status == g.GPD_ERR_ARG
    out = cp.plan.empty(g.GPD_Q_OUT_ELEMS_BWD)
    with pytest.raises(g.GpdError) as ei:
        g.gpd_worker_gemm(cp.plan, g.GPD_BWD, cp.W_shares, Xs, out)
    assert ei.value.status == g.GPD_ERR_UNSUPPORTED
    with pytest.raises(g.GpdError) as ei:
        g.gpd_locate_errors(cp.plan, g.GPD_AUDIT, cp.W_shares, cp.res, cp.ws)
    assert ei.value.status == g.GPD_ERR_UNSUPPORTED
    with pytest.raises(g.GpdError) as ei:
        g.gpd_regenerate_shares(cp.plan, cp.W_shares, cp.res, cp.ws)
    assert ei.value.status == g.GPD_ERR_UNSUPPORTED


# --------------------------------------------------------------------------------------------------
# training mode: every product of the coded step on digit planes, FP64 shares kept beside them
# --------------------------------------------------------------------------------------------------
def _pair_tolerance(rowmax_a, rowmax_b, K, slack_a=1.0, slack_b=1.0):
    """Per-entry bound for A B^T from the largest magnitudes of A's and B's operand rows (scales lie
    within 4.07 times those, times `slack` where the scale comes from a bound instead)."""
    return 4.0 * np.sqrt(K) * PER_TERM[6] * (SCALE_OVER_MAX * slack_a * rowmax_a)[:, :, None] * \
        (SCALE_OVER_MAX * slack_b * rowmax_b)[:, None, :]


@pytest.mark.parametrize("N1,N0,B,m,n,P", [
    (512, 256, 128, 2, 2, 10),          # whole tiles; thresholds 5 / 6 / 4
    (416, 320, 48, 2, 4, 14),           # ragged tiles: 208-row and 80-column shares, batch 48; thresholds 11 / 12 / 8
    (256, 128, 64, 4, 4, 36),           # the autoencoder's code: thresholds 19 / 28 / 16
])
def test_training_mode_products_update_and_audit_match_oracle(N1, N0, B, m, n, P):
    rng = np.random.default_rng(N1 + N0 + B)
    W = (rng.standard_normal((N1, N0)) / np.sqrt(N0)).astype(np.float32)
    X = rng.standard_normal((N0, B)).astype(np.float32)
    DT = (rng.standard_normal((B, N1)) / B).astype(np.float32)
    Delta = np.ascontiguousarray(DT.T)
    code = GPCode(N1, N0, B, m, n, 1, 1, P)
    cp = CodedProduct(code, precision=g.GPD_PREC_FP64_SLICED_TRAIN)
    assert cp.plan.query(g.GPD_Q_PRECISION) == g.GPD_PREC_FP64_SLICED_TRAIN and cp.np_dtype == np.float64
    M, K = N1 // m, N0 // n
    Wsh = cp.encode_W(W)
    assert Wsh.numel() > P * M * K                                 # FP64 shares plus the two sliced copies
    Ws_o = op.encode_W(W, code)
    master = host(Wsh)[:P * M * K].reshape(P, M, K)
    assert np.abs(master - Ws_o).max() <= 4e-16 * np.abs(Ws_o).max() * m * n
    # forward product: rows of W~_p (exact row maxima) x columns of X~_p
    Xs_o = op.encode_X(X, code)
    Z = cp.outputs_as_array(g.GPD_FWD, cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X)))
    Zo = op.worker_products(Ws_o, Xs_o)
    tol = _pair_tolerance(np.abs(Ws_o).max(axis=2), np.abs(Xs_o).max(axis=1), K)
    assert np.isfinite(Z).all() and (np.abs(Z - Zo) <= tol).all(), float((np.abs(Z - Zo) / tol).max())
    # backward product: rows of Delta~^T_p (scale from the bound over its m blocks) x columns of W~_p
    Ds_o = op.encode_DeltaT(DT, code)
    Zb_t = cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT))
    Zb = cp.outputs_as_array(g.GPD_BWD, Zb_t)
    Zbo = op.worker_products(Ds_o, Ws_o)
    blk = np.abs(DT.astype(np.float64)).reshape(B, m, M).max(axis=2)                        # [B][m]
    bound = np.einsum("pi,bi->pb", np.abs(code.points)[:, None] ** code.exp_DeltaT()[0][None, :], blk)
    tol = _pair_tolerance(bound, np.abs(Ws_o).max(axis=1), M)
    assert np.isfinite(Zb).all() and (np.abs(Zb - Zbo) <= tol).all(), float((np.abs(Zb - Zbo) / tol).max())
    # the backward outputs go through location and decoding like any others
    nodes = np.zeros(P, dtype=bool)
    nodes[[1, P - 2][:min(2, P - code.Q_b - 1)]] = True             # as many as the backward product can correct
    mask = sum(1 << int(q) for q in np.flatnonzero(nodes))
    g.gpd_inject(cp.plan, g.GPD_BWD, Zb_t, 21, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=mask, scale=1.0)
    Zr = Zbo.copy()
    oinj.inject_gauss(Zr, 21, 1.0, nodes=nodes)
    ro = locate_subspace(Zr, code.points, code.Q_b, tolerances_for(np.float64))
    r = cp.locate(g.GPD_BWD, Zb_t)
    assert r.outcome == ro.outcome == CORRECTED and np.array_equal(cp.flags(r), ro.flagged) and np.array_equal(ro.flagged, nodes)
    CT = cp.decode(g.GPD_BWD, Zb_t)
    assert op.rel_fro(CT, op.ref_backward(DT, W)) < 1e-4
    assert op.rel_fro(CT, op.decode(Zr, code, BWD, use=~ro.flagged)) < 1e-4
    # coded update with weight decay (Eq. 10): FP64 shares, then audit through the re-cut copies' source
    eta, lam = 0.0625, 0.125
    Dh_o, Xh_o = op.encode_update_operands(Delta, X, code)
    g.gpd_update_shares(cp.plan, Wsh, cp.encode(g.GPD_OPERAND_DELTA_UPD, Delta), cp.encode(g.GPD_OPERAND_X_UPD, X), eta, lam)
    want = op.update_shares(Ws_o, Dh_o, Xh_o, eta=eta, lam=lam)
    got = host(Wsh)[:P * M * K].reshape(P, M, K)
    dmax = np.einsum("pi,ri->pr", np.abs(code.points)[:, None] ** code.exp_update()[0][None, :],
                     np.abs(Delta.astype(np.float64)).reshape(m, M, B).max(axis=2).T)       # bound of |Delta^_p| rows
    xmax = np.einsum("pj,rj->pr", np.abs(code.points)[:, None] ** code.exp_update()[1][None, :],
                     np.abs(X.astype(np.float64)).reshape(n, K, B).max(axis=2).T)
    tol = eta * _pair_tolerance(dmax, xmax, B) + 4e-16 * np.abs(want).max()
    assert (np.abs(got - want) <= tol).all(), float((np.abs(got - want) / tol).max())
    r = cp.locate(g.GPD_AUDIT, Wsh)
    assert r.outcome == NO_ERROR
    assert op.rel_fro(cp.decode(g.GPD_AUDIT, Wsh), op.ref_update(W, Delta, X, eta, lam)) < 1e-4
    # the forward product after the update reads the re-cut row copy: it must see the new shares
    Z2 = cp.outputs_as_array(g.GPD_FWD, cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X)))
    Z2o = op.worker_products(want, Xs_o)
    tol = _pair_tolerance(np.abs(want).max(axis=2), np.abs(Xs_o).max(axis=1), K)
    assert (np.abs(Z2 - Z2o) <= tol).all()
    # and so must the backward product (column copy)
    Zb2 = cp.outputs_as_array(g.GPD_BWD, cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT)))
    tol = _pair_tolerance(bound, np.abs(want).max(axis=1), M)
    assert (np.abs(Zb2 - op.worker_products(Ds_o, want)) <= tol).all()
    # share errors: written into the FP64 shares, seen by the next forward product, repaired by regeneration
    g.gpd_inject(cp.plan, g.GPD_AUDIT, Wsh, 22, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=1 << 3, scale=0.1)
    Zf_t = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    r = cp.locate(g.GPD_FWD, Zf_t)
    assert r.outcome == CORRECTED and list(np.flatnonzero(cp.flags(r))) == [3]
    g.gpd_regenerate_shares(cp.plan, Wsh, cp.res, cp.ws)
    got = host(Wsh)[:P * M * K].reshape(P, M, K)
    assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
    Z3 = cp.outputs_as_array(g.GPD_FWD, cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X)))
    assert np.abs(Z3 - Z2o).max() <= 1e-10 * np.sqrt(np.mean(Z2o ** 2))
    # an update gated by a failed decode of the backward product changes nothing: neither the FP64 shares
    # nor the two sliced copies (the forward and the backward product read them)
    gate = g.new_results(1)
    gate.view(torch.int32)[0] = g.GPD_DECODE_FAILURE
    before = host(Wsh).copy()
    Zb3 = cp.outputs_as_array(g.GPD_BWD, cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT)))
    g.gpd_update_shares(cp.plan, Wsh, cp.encode(g.GPD_OPERAND_DELTA_UPD, Delta), cp.encode(g.GPD_OPERAND_X_UPD, X),
                        eta, lam, gate=gate)
    assert np.array_equal(host(Wsh)[:P * M * K], before[:P * M * K])
    assert np.array_equal(cp.outputs_as_array(g.GPD_FWD, cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))), Z3)
    assert np.array_equal(cp.outputs_as_array(g.GPD_BWD, cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT))), Zb3)
    assert g.gpd_device_status() == 0


def test_training_mode_rejects_shapes_it_cannot_serve():
    # N1/m = 40 is not a multiple of 16 (backward contraction length)
    with pytest.raises(g.GpdError) as ei:
        g.gpd_plan((80, 64, 32), (2, 2, 1, 1), 10, precision=g.GPD_PREC_FP64_SLICED_TRAIN)
    assert ei.value.status == g.GPD_ERR_UNSUPPORTED
    # a forward-only plan (P below the backward threshold) has no use for it
    with pytest.raises(g.GpdError) as ei:
        g.gpd_plan((96, 64, 48), (3, 2, 1, 3), 9, precision=g.GPD_PREC_FP64_SLICED_TRAIN)
    assert ei.value.status in (g.GPD_ERR_UNSUPPORTED, g.GPD_ERR_P_TOO_SMALL)
