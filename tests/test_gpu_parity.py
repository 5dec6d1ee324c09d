"""GPU parity: every stage of the CUDA path against the CPU FP64 oracle, through the C ABI.

Bars: integer / index work (error-location outcome, flag vectors, bit flips, which entries an
injector touches) bit-exact; decoded floating point within 1e-4 relative Frobenius error (the
target the workloads state); intermediate FP64 quantities much tighter, as written per test.
"""

import itertools

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():                       # collected on a CPU machine: nothing to run
    pytest.skip("needs a CUDA device", allow_module_level=True)

import paper_1811_10751_b200 as g                        # noqa: E402
import workloads as wl                                   # noqa: E402
from oracle import inject as oinj                        # noqa: E402
from oracle import product as op                         # noqa: E402
from oracle.code import GPCode, FWD, BWD, AUDIT          # noqa: E402
from oracle.locate import (CORRECTED, DECODE_FAILURE, NO_ERROR, locate_subspace,  # noqa: E402
                           tolerances_for)
from tests.gpu_pipeline import CodedProduct, dev, host, make_code   # noqa: E402

REL_TOL = 1e-4                                           # decoded outputs, relative Frobenius


def rms(a):
    return float(np.sqrt(np.mean(np.asarray(a, dtype=np.float64) ** 2)))


def rand(shape, seed, dist="gauss"):
    r = np.random.default_rng(seed)
    a = r.standard_normal(shape) if dist == "gauss" else r.uniform(-1, 1, shape)
    return a.astype(np.float32)


# --------------------------------------------------------------------------------------------------
# encode
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N1,N0,B,m,n,d1,d2,P,prec", [
    (64, 64, 64, 2, 2, 2, 1, 11, g.GPD_PREC_FP32),
    (512, 1024, 128, 2, 4, 2, 1, 25, g.GPD_PREC_FP64),
    (96, 60, 6, 3, 2, 2, 3, 20, g.GPD_PREC_FP64),            # block widths not multiples of 4
    (10, 4096, 256, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),        # 5-row blocks
    (4096, 4096, 1, 4, 2, 1, 1, 13, g.GPD_PREC_FP32),        # matrix-vector
    (256, 128, 64, 4, 4, 1, 1, 36, g.GPD_PREC_FP64),
])
def test_encode_matches_oracle(N1, N0, B, m, n, d1, d2, P, prec):
    code = GPCode(N1, N0, B, m, n, d1, d2, P)
    cp = CodedProduct(code, prec)
    W, X, DT = rand((N1, N0), 1), rand((N0, B), 2), rand((B, N1), 3)
    f32 = cp.np_dtype == np.float32
    rtol = 2e-7 if f32 else 1e-14
    cases = [(cp.encode_W(W), op.encode_W(W, code)),
             (cp.encode(g.GPD_OPERAND_X_FWD, X), op.encode_X(X, code))]
    if P >= code.Q_b:
        cases.append((cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT), op.encode_DeltaT(DT, code)))
    Dh, Xh = op.encode_update_operands(DT.T.copy(), X, code)
    cases.append((cp.encode(g.GPD_OPERAND_DELTA_UPD, DT.T.copy()), Dh))
    cases.append((cp.encode(g.GPD_OPERAND_X_UPD, X), Xh))
    for got, want in cases:
        got = host(got).reshape(want.shape).astype(np.float64)
        scale = np.abs(want).max()
        assert np.abs(got - want).max() <= rtol * scale * 4


# --------------------------------------------------------------------------------------------------
# worker products and coded update
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N1,N0,B,m,n,d1,d2,P,prec", [
    (512, 512, 256, 2, 2, 2, 2, 16, g.GPD_PREC_FP64),        # tensor-core FP64 tiles, exact multiples
    (400, 200, 144, 2, 2, 2, 2, 16, g.GPD_PREC_FP64),        # ragged tails in M, N and K
    (66, 50, 14, 2, 2, 2, 2, 16, g.GPD_PREC_FP64),           # odd sizes -> CUDA-core kernel
    (512, 512, 256, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),        # tcgen05 3xTF32 tiles, exact multiples
    (400, 272, 200, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),        # tcgen05 path with ragged M, N and K
    (2048, 1024, 256, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),      # many k-blocks: the stage ring wraps; 160 tiles on 148
                                                             # SMs: the 12 left over are cut into four parts of K
    (600, 1024, 200, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),       # 60 ragged tiles (300 x 200 per node), each cut into two
                                                             # parts of K = 512 whose sums meet in the plan's scratch
    (512, 768, 1000, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),       # mini-batch 1000: the update's contraction spans four
                                                             # accumulation groups (the last one short)
    (10, 512, 64, 2, 2, 1, 1, 10, g.GPD_PREC_FP32),          # 5-row blocks
    (1024, 512, 1, 4, 2, 1, 1, 13, g.GPD_PREC_FP32),         # matrix-vector
    (1024, 512, 1, 4, 2, 1, 1, 13, g.GPD_PREC_FP64),
])
def test_worker_products_and_update_match_oracle(N1, N0, B, m, n, d1, d2, P, prec):
    code = GPCode(N1, N0, B, m, n, d1, d2, P)
    cp = CodedProduct(code, prec)
    W, X, DT = rand((N1, N0), 4), rand((N0, B), 5), rand((B, N1), 6)
    f32 = cp.np_dtype == np.float32

    def check(got, want):
        # Against the FP64 product of the same stored shares, relative to the rms of the outputs.
        # FP64 paths: a few ulp of the accumulated magnitude.  FP32 paths (tensor-core 3xTF32 with
        # accumulation chains cut every 64 elements of K, or FP32 FMA loops): measured 4.7e-7 rms and
        # 4.4e-6 worst entry at K = 2048; the bounds are four times that.
        err = np.asarray(got, dtype=np.float64) - want
        assert np.isfinite(got).all()
        if f32:
            assert rms(err) <= 2e-6 * rms(want) and np.abs(err).max() <= 2e-5 * rms(want)
        else:
            assert np.abs(err).max() <= 8e-13 * rms(want)

    Wsh = cp.encode_W(W)
    Ws_o = host(Wsh).reshape(P, N1 // m, N0 // n).astype(np.float64)      # same stored shares
    Xsh = cp.encode(g.GPD_OPERAND_X_FWD, X)
    Z = cp.outputs_as_array(g.GPD_FWD, cp.products(g.GPD_FWD, Xsh))
    want = op.worker_products(Ws_o, host(Xsh).reshape(P, N0 // n, B // d1).astype(np.float64))
    check(Z, want)
    if P >= code.Q_b:
        Dsh = cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT)
        Zb = cp.outputs_as_array(g.GPD_BWD, cp.products(g.GPD_BWD, Dsh))
        want = op.worker_products(host(Dsh).reshape(P, B // d2, N1 // m).astype(np.float64), Ws_o)
        check(Zb, want)
    # coded update in place, with weight decay
    Delta = DT.T.copy()
    Dh, Xh = cp.encode(g.GPD_OPERAND_DELTA_UPD, Delta), cp.encode(g.GPD_OPERAND_X_UPD, X)
    want = op.update_shares(Ws_o, host(Dh).reshape(P, N1 // m, B).astype(np.float64),
                            host(Xh).reshape(P, N0 // n, B).astype(np.float64), eta=0.0625, lam=0.125)
    g.gpd_update_shares(cp.plan, Wsh, Dh, Xh, 0.0625, 0.125)      # both exact in FP32: the call takes floats
    got = host(Wsh).reshape(want.shape).astype(np.float64)
    # new share = shrink * old + eta * (Delta^ X^^T): one rounding of the stored result (2 ulp allowed)
    # plus eta times the error of the product (bounded as above; the update's chains are up to 256 long:
    # measured 1.8e-6 rms, 1.5e-5 worst entry of the product's rms)
    inc = (want - (1.0 - 0.0625 * 0.125) * Ws_o) / 0.0625
    ulp = 2.0 ** -23 if f32 else 2.0 ** -52
    prod_err = 6e-5 if f32 else 8e-13
    assert np.abs(got - want).max() <= 2 * ulp * np.abs(want).max() + 0.0625 * prod_err * rms(inc)
    assert g.gpd_device_status() == 0                        # no bounded wait expired on the tensor path


# --------------------------------------------------------------------------------------------------
# injection: same clean buffer on both sides
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("prec", [g.GPD_PREC_FP32, g.GPD_PREC_FP64])
def test_injectors_match_oracle(prec):
    code = GPCode(96, 64, 40, 2, 2, 2, 1, 14)
    cp = CodedProduct(code, prec)
    L = (96 // 2) * (40 // 2)
    clean = np.random.default_rng(7).standard_normal((14, L)).astype(cp.np_dtype)
    hit = torch.zeros(1, dtype=torch.int64, device="cuda")

    def mask_of(h):
        return np.array([(int(h.item()) >> p) & 1 for p in range(14)], dtype=bool)

    for seed in (1, 2, 3):
        Z = dev(clean)
        g.gpd_inject(cp.plan, g.GPD_FWD, Z, seed, g.GPD_INJECT_BITFLIP, count=3, scale=1.0, hit_mask=hit)
        ref = clean.copy()
        sel = oinj.inject_bitflip(ref, seed, 3, 1.0)
        itype = np.uint32 if prec == g.GPD_PREC_FP32 else np.uint64
        assert np.array_equal(host(Z).view(itype), ref.view(itype))            # bit-exact
        assert np.array_equal(mask_of(hit), sel)

        Z = dev(clean)
        g.gpd_inject(cp.plan, g.GPD_FWD, Z, seed, g.GPD_INJECT_ADDITIVE, prob=0.3, scale=2.0, hit_mask=hit)
        ref = clean.copy()
        sel = oinj.inject_additive(ref, seed, 2.0, prob=0.3)
        assert np.array_equal(host(Z).view(itype), ref.view(itype))            # bit-exact
        assert np.array_equal(mask_of(hit), sel)

        Z = dev(clean)
        nodes = np.zeros(14, dtype=bool)
        nodes[[2, 9]] = True
        g.gpd_inject(cp.plan, g.GPD_FWD, Z, seed, g.GPD_INJECT_GAUSS, prob=-1.0,
                     node_mask=(1 << 2) | (1 << 9), scale=1.5, hit_mask=hit)
        ref = clean.copy()
        oinj.inject_gauss(ref, seed, 1.5, nodes=nodes)
        assert np.array_equal(mask_of(hit), nodes)
        assert np.array_equal(host(Z)[~nodes], clean[~nodes])
        tol = 1e-6 if prec == g.GPD_PREC_FP32 else 1e-12
        assert np.abs(host(Z).astype(np.float64) - ref.astype(np.float64)).max() < tol * 8


# --------------------------------------------------------------------------------------------------
# config 1: tiny matmul, no errors, every threshold-sized subset
# --------------------------------------------------------------------------------------------------
def test_config1_all_subsets():
    cfg = wl.CONFIG_1_TINY
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code)
    assert cp.np_dtype == np.float32
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    r = cp.locate(g.GPD_FWD, Z)
    assert r.outcome == NO_ERROR and r.n_flagged == 0 and r.n_active == 0
    ref = op.ref_forward(W, X)
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    assert op.rel_fro(cp.decode(g.GPD_FWD, Z), ref) < REL_TOL
    worst = 0.0
    for keep in itertools.combinations(range(cfg.P), code.Q_f):
        use = np.zeros(cfg.P, dtype=bool)
        use[list(keep)] = True
        S = cp.decode(g.GPD_FWD, Z, use_mask=use)
        worst = max(worst, op.rel_fro(S, ref))
        assert op.rel_fro(S, op.decode(Zo, code, FWD, use)) < REL_TOL
    assert worst < REL_TOL


# --------------------------------------------------------------------------------------------------
# config 2: matrix-vector with two bit flips (full size)
# --------------------------------------------------------------------------------------------------
def test_config2_matvec_two_bitflips():
    cfg = wl.CONFIG_2_MATVEC
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    ref = op.ref_forward(W, X)
    # oracle pipeline on its own outputs
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code)).astype(np.float32)
    scale = rms(Zo)
    for seed in cfg.inject_seeds + (5, 6, 7):
        Zg = Z.clone()
        hit = torch.zeros(1, dtype=torch.int64, device="cuda")
        g.gpd_inject(cp.plan, g.GPD_FWD, Zg, seed, g.GPD_INJECT_BITFLIP, count=cfg.inject_count, scale=scale,
                     hit_mask=hit)
        Zr = Zo.copy()
        sel = oinj.inject_bitflip(Zr, seed, cfg.inject_count, scale)
        ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float32))
        r = cp.locate(g.GPD_FWD, Zg)
        assert r.outcome == ro.outcome == CORRECTED
        assert np.array_equal(cp.flags(r), ro.flagged) and np.array_equal(ro.flagged, sel)
        assert sel.sum() == 2 and r.n_flagged == 2
        S = cp.decode(g.GPD_FWD, Zg)
        assert op.rel_fro(S, ref) < REL_TOL
        assert op.rel_fro(S, op.decode(Zr, code, FWD, use=~ro.flagged)) < REL_TOL


def test_config2_two_bitflips_in_one_position():
    """Both flips at the same output position: one failing codeword, a rank-1 syndrome Gram matrix
    and two erroneous nodes.  floor((13 - 9) / 2) = 2 errors in one codeword are correctable
    (adversarial-model lemma); the locator gets there through its search over supersets."""
    cfg = wl.CONFIG_2_MATVEC
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code)).astype(np.float32).reshape(cfg.P, -1)
    L = Zo.shape[1]
    ref = op.ref_forward(W, X)
    for (pa, ba), (pb, bb), pos in (((2, 27), (11, 22), 100), ((0, 30), (12, 25), 1023), ((5, 24), (6, 29), 0)):
        Zg, Zr = Z.clone(), Zo.copy()
        for p, bit in ((pa, ba), (pb, bb)):
            Zr.view(np.uint32)[p, pos] ^= np.uint32(1 << bit)
            word = Zg.view(torch.int32)[p * L + pos]
            Zg.view(torch.int32)[p * L + pos] = word ^ (1 << bit)
        ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float32))
        r = cp.locate(g.GPD_FWD, Zg)
        assert r.outcome == ro.outcome == CORRECTED, (r.outcome, ro.outcome)
        assert np.array_equal(cp.flags(r), ro.flagged) and sorted(np.flatnonzero(ro.flagged)) == sorted((pa, pb))
        assert r.rank == ro.rank == 1 and r.n_active == ro.n_active == 1
        assert op.rel_fro(cp.decode(g.GPD_FWD, Zg), ref) < REL_TOL


def test_rank_deficient_patterns_small_code():
    """A single codeword per node (L = 1) and two (L = 2): every support of up to P-Q errors; the
    decision (outcome, flags) is the oracle's for each of them, failures included."""
    for P, B in ((9, 1), (10, 2)):                                # threshold 5; L = B positions per node
        m, n, d1 = 2, 2, 1
        N1, N0 = m, 3 * n                                             # one-row blocks of W
        code = GPCode(N1, N0, B, m, n, d1, 1, P)
        cp = CodedProduct(code, g.GPD_PREC_FP64)
        W, X = rand((N1, N0), 91), rand((N0, B), 92)
        cp.encode_W(W)
        Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
        Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code)).reshape(P, -1)
        Lp = Zo.shape[1]
        rng = np.random.default_rng(93)
        R = P - code.Q_f
        for size in range(1, R + 1):
            for nodes in itertools.combinations(range(P), size):
                e = rng.uniform(0.5, 2.0, (size, Lp)) * rng.choice([-1.0, 1.0], (size, Lp))
                Zr = Zo.copy()
                Zr[list(nodes)] += e
                Zg = Z.clone().reshape(P, Lp)
                Zg[list(nodes)] += dev(e)
                ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
                r = cp.locate(g.GPD_FWD, Zg.reshape(-1))
                assert r.outcome == ro.outcome, (nodes, r.outcome, ro.outcome)
                assert np.array_equal(cp.flags(r), ro.flagged), nodes
                assert ro.outcome == (CORRECTED if size < R else DECODE_FAILURE)


def test_huge_finite_values_are_flagged():
    """FP64 outputs: flipping exponent bit 62 of a value below 1 multiplies it by 2^1024 - finite, but
    its square is not.  Such a value is handled like a non-finite one (node flagged up front)."""
    cfg = wl.scaled_down(wl.CONFIG_3_MATMUL, 16)
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code)
    assert cp.np_dtype == np.float64
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    ref = op.ref_forward(W, X)
    Zr = op.worker_products(op.encode_W(W, code), op.encode_X(X, code)).reshape(cfg.P, -1)
    L = Zr.shape[1]
    pos = int(np.flatnonzero(np.abs(Zr[6]) < 1.0)[3])
    Zr.view(np.uint64)[6, pos] ^= np.uint64(1 << 62)
    Zg = Z.clone()
    Zg.view(torch.int64)[6 * L + pos] ^= (1 << 62)
    assert np.isfinite(Zr[6, pos]) and abs(Zr[6, pos]) > 2.0 ** 900
    planted = float(host(Zg).reshape(cfg.P, L)[6, pos])
    assert np.isfinite(planted) and abs(planted) > 2.0 ** 900
    ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
    r = cp.locate(g.GPD_FWD, Zg)
    assert r.outcome == ro.outcome == CORRECTED
    assert np.array_equal(cp.flags(r), ro.flagged) and list(np.flatnonzero(ro.flagged)) == [6]
    assert np.array_equal(np.array(list(r.forced)[:cfg.P], dtype=bool), ro.forced) and ro.forced[6]
    S = cp.decode(g.GPD_FWD, Zg)
    assert np.isfinite(S).all() and op.rel_fro(S, ref) < REL_TOL
    # per-position correction: the position is reported as failed and left untouched on both sides
    from oracle.perpos import correct_positions
    rp_o = correct_positions(Zr, code.points, code.Q_f, tolerances_for(np.float64))
    Zp = Zg.clone()
    rp = g.gpd_correct_positions(cp.plan, g.GPD_FWD, Zp)
    assert rp.outcome == rp_o.outcome == DECODE_FAILURE
    assert (rp.n_active, rp.n_failed, rp.n_corrected) == (rp_o.n_active, rp_o.n_failed, rp_o.n_corrected) == (1, 1, 0)
    assert torch.equal(Zp.view(torch.int64), Zg.view(torch.int64))


# --------------------------------------------------------------------------------------------------
# threshold 9 through the tensor-core FP32 path: the largest threshold for which a plan keeps FP32
# shares, at a size where the 128 x 128 tcgen05 tiles (not the small-block kernel) do the products
# --------------------------------------------------------------------------------------------------
def test_threshold9_on_the_tensor_core_fp32_path():
    N1, N0, B, P = 4096, 4096, 512, 11
    rng = np.random.default_rng(181110760)
    W = (rng.standard_normal((N1, N0)) / np.sqrt(N0)).astype(np.float32)
    X = rng.standard_normal((N0, B)).astype(np.float32)
    code = GPCode(N1, N0, B, 2, 2, 2, 1, P)
    assert code.Q_f == 9
    cp = CodedProduct(code)                                   # GPD_PREC_AUTO
    assert cp.np_dtype == np.float32
    Wsh = cp.encode_W(W)
    Xsh = cp.encode(g.GPD_OPERAND_X_FWD, X)
    Z = cp.products(g.GPD_FWD, Xsh)
    ref = op.ref_forward(W, X)
    # worker products against FP64 products of the same stored shares: the tensor-core accumulation
    # chain is cut every 128 elements of K, measured 9e-7 of the output rms (an FP32 FMA loop: 2e-7)
    want = op.worker_products(host(Wsh).reshape(P, N1 // 2, N0 // 2), host(Xsh).reshape(P, N0 // 2, B // 2))
    err = cp.outputs_as_array(g.GPD_FWD, Z) - want
    assert rms(err) <= 4e-6 * rms(want) and np.abs(err).max() <= 4e-5 * rms(want)
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    # clean: every node; the two end nodes dropped (the worst conditioned nine-subset family)
    r = cp.locate(g.GPD_FWD, Z)
    assert r.outcome == NO_ERROR and r.n_active == 0
    S = cp.decode(g.GPD_FWD, Z)
    assert op.rel_fro(S, ref) < REL_TOL / 3 and op.rel_fro(S, op.decode(Zo, code, FWD)) < REL_TOL / 3
    for drop in ((0, 10), (0, 1), (9, 10)):
        use = np.ones(P, dtype=bool)
        use[list(drop)] = False
        Sd = cp.decode(g.GPD_FWD, Z, use_mask=use)
        assert op.rel_fro(Sd, ref) < REL_TOL and op.rel_fro(Sd, op.decode(Zo, code, FWD, use)) < REL_TOL
    # one erroneous node (Error Model 2)
    nodes = np.zeros(P, dtype=bool)
    nodes[4] = True
    Zg = Z.clone()
    g.gpd_inject(cp.plan, g.GPD_FWD, Zg, 7, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=1 << 4, scale=1.0)
    Zr = Zo.astype(np.float32)
    oinj.inject_gauss(Zr, 7, 1.0, nodes=nodes)
    ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float32))
    r = cp.locate(g.GPD_FWD, Zg)
    assert r.outcome == ro.outcome == CORRECTED and np.array_equal(cp.flags(r), ro.flagged)
    assert np.array_equal(ro.flagged, nodes)
    S = cp.decode(g.GPD_FWD, Zg)
    assert op.rel_fro(S, ref) < REL_TOL / 2
    assert op.rel_fro(S, op.decode(Zr, code, FWD, use=~ro.flagged)) < REL_TOL / 2
    assert g.gpd_device_status() == 0


# --------------------------------------------------------------------------------------------------
# config 3 at reduced size: additive errors on random nodes, several seeds, failure included
# --------------------------------------------------------------------------------------------------
def _run_additive_case(cfg, seeds, precision=g.GPD_PREC_AUTO):
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code, precision=precision)
    assert cp.np_dtype == np.float64
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    ref = op.ref_forward(W, X)
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    scale = rms(Zo)
    outcomes = []
    for seed in seeds:
        Zg = Z.clone()
        g.gpd_inject(cp.plan, g.GPD_FWD, Zg, seed, g.GPD_INJECT_ADDITIVE, prob=cfg.inject_prob, scale=scale)
        Zr = Zo.copy()
        sel = oinj.inject_additive(Zr, seed, scale, prob=cfg.inject_prob)
        ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
        r = cp.locate(g.GPD_FWD, Zg)
        assert r.outcome == ro.outcome, (seed, r.outcome, ro.outcome, sel.sum())
        assert np.array_equal(cp.flags(r), ro.flagged)
        outcomes.append(r.outcome)
        S = cp.decode(g.GPD_FWD, Zg, fill=-7.0)
        if r.outcome == DECODE_FAILURE:
            assert (S == -7.0).all()                                   # nothing written
            continue
        assert np.array_equal(ro.flagged, sel)
        assert op.rel_fro(S, ref) < REL_TOL
        assert op.rel_fro(S, op.decode(Zr, code, FWD, use=~ro.flagged)) < REL_TOL
    return outcomes


@pytest.mark.parametrize("precision", [g.GPD_PREC_AUTO, g.GPD_PREC_FP64_SLICED, g.GPD_PREC_FP64_SLICED40])
def test_config3_scaled_additive_errors(precision):
    cfg = wl.scaled_down(wl.CONFIG_3_MATMUL, 8)                         # 1024 x 1024 x 64, same code
    outcomes = _run_additive_case(cfg, cfg.inject_seeds, precision)
    assert CORRECTED in outcomes


def test_too_many_errors_is_a_declared_failure():
    cfg = wl.scaled_down(wl.CONFIG_3_MATMUL, 16)
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    for n_bad in (6, 9):                                                # P - Q = 6: budget is 5
        mask = sum(1 << p for p in range(0, 2 * n_bad, 2))
        nodes = np.array([(mask >> p) & 1 for p in range(cfg.P)], dtype=bool)
        Zg = Z.clone()
        g.gpd_inject(cp.plan, g.GPD_FWD, Zg, 11, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=mask, scale=1.0)
        Zr = Zo.copy()
        oinj.inject_gauss(Zr, 11, 1.0, nodes=nodes)
        ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
        r = cp.locate(g.GPD_FWD, Zg)
        assert r.outcome == ro.outcome == DECODE_FAILURE
        S = cp.decode(g.GPD_FWD, Zg, fill=3.0)
        assert (S == 3.0).all()


def test_erasures_and_nonfinite_values():
    cfg = wl.scaled_down(wl.CONFIG_3_MATMUL, 16)
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    ref = op.ref_forward(W, X)
    Zg = Z.clone()
    L = Zg.numel() // cfg.P
    Zg[3 * L + 17] = float("inf")
    Zg[20 * L + 5] = float("nan")
    erased = np.zeros(cfg.P, dtype=bool)
    erased[[7, 8]] = True
    r = cp.locate(g.GPD_FWD, Zg, erased=erased)
    # the oracle works on its own outputs, with the same two values planted
    Zr = op.worker_products(op.encode_W(W, code), op.encode_X(X, code)).reshape(cfg.P, L)
    Zr[3, 17] = np.inf
    Zr[20, 5] = np.nan
    ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64), erased=erased)
    assert r.outcome == ro.outcome == CORRECTED
    assert np.array_equal(cp.flags(r), ro.flagged)
    assert sorted(np.flatnonzero(ro.flagged)) == [3, 7, 8, 20]
    assert np.array_equal(np.array(list(r.forced)[:cfg.P], dtype=bool), ro.forced)
    assert op.rel_fro(cp.decode(g.GPD_FWD, Zg), ref) < REL_TOL


# --------------------------------------------------------------------------------------------------
# backward product and audit of the shares
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N1,N0,B,m,n,d2,P,prec", [
    (512, 512, 64, 2, 2, 1, 10, g.GPD_PREC_AUTO),              # FP32 path (thresholds 5/6/4)
    (256, 512, 128, 4, 4, 1, 36, g.GPD_PREC_AUTO),             # FP64 path (thresholds 19/28/16)
    (128, 96, 24, 2, 3, 3, 24, g.GPD_PREC_AUTO),               # d2 = 3: Q_b = 21
])
def test_backward_and_audit(N1, N0, B, m, n, d2, P, prec):
    code = GPCode(N1, N0, B, m, n, 1, d2, P)
    cp = CodedProduct(code, prec)
    W, DT = (rand((N1, N0), 8) / np.sqrt(N0)).astype(np.float32), rand((B, N1), 9)
    Wsh = cp.encode_W(W)
    Dsh = cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT)
    Z = cp.products(g.GPD_BWD, Dsh)
    nodes = np.zeros(P, dtype=bool)
    nodes[[1, P - 2]] = True
    g.gpd_inject(cp.plan, g.GPD_BWD, Z, 21, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=(1 << 1) | (1 << (P - 2)),
                 scale=1.0)
    r = cp.locate(g.GPD_BWD, Z)
    Zr = op.worker_products(op.encode_DeltaT(DT, code), op.encode_W(W, code)).astype(cp.np_dtype)
    oinj.inject_gauss(Zr, 21, 1.0, nodes=nodes)
    ro = locate_subspace(Zr, code.points, code.Q_b, tolerances_for(cp.np_dtype))
    assert r.outcome == ro.outcome == CORRECTED and np.array_equal(cp.flags(r), ro.flagged)
    assert np.array_equal(ro.flagged, nodes)
    CT = cp.decode(g.GPD_BWD, Z)
    assert op.rel_fro(CT, op.ref_backward(DT, W)) < REL_TOL
    assert op.rel_fro(CT, op.decode(Zr, code, BWD, use=~ro.flagged)) < REL_TOL
    # audit: corrupt one stored share, find it, read W back
    g.gpd_inject(cp.plan, g.GPD_AUDIT, Wsh, 22, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=1 << 4, scale=0.1)
    r = cp.locate(g.GPD_AUDIT, Wsh)
    assert r.outcome == CORRECTED and list(np.flatnonzero(cp.flags(r))) == [4]
    assert op.rel_fro(cp.decode(g.GPD_AUDIT, Wsh), W) < REL_TOL


# --------------------------------------------------------------------------------------------------
# config 4, one full-size hidden layer (4096 x 4096, batch 256): forward, backward, update on the
# tensor-core FP32 path, with Gaussian node errors; decoded outputs against the FP64 products
# --------------------------------------------------------------------------------------------------
def test_config4_full_size_layer():
    c4 = wl.CONFIG_4_MLP
    N, B, P = c4.widths[1], c4.B, c4.P
    rng = np.random.default_rng(c4.seed)
    W = (rng.standard_normal((N, N)) * np.sqrt(2.0 / N)).astype(np.float32)
    X = np.maximum(rng.standard_normal((N, B)), 0).astype(np.float32)             # a ReLU output
    Delta = (rng.standard_normal((N, B)) / B).astype(np.float32)
    DT = np.ascontiguousarray(Delta.T)
    code = GPCode(N, N, B, c4.m, c4.n, 1, 1, P)
    cp = CodedProduct(code)
    assert cp.np_dtype == np.float32
    Wsh = cp.encode_W(W)
    nodes_f, nodes_b = (1 << 0) | (1 << 6), 1 << 9
    Zf = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    g.gpd_inject(cp.plan, g.GPD_FWD, Zf, 41, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=nodes_f, scale=1.0)
    r = cp.locate(g.GPD_FWD, Zf)
    assert r.outcome == CORRECTED and list(np.flatnonzero(cp.flags(r))) == [0, 6]
    S = cp.decode(g.GPD_FWD, Zf)
    assert op.rel_fro(S, op.ref_forward(W, X)) < REL_TOL
    Zb = cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT))
    g.gpd_inject(cp.plan, g.GPD_BWD, Zb, 42, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=nodes_b, scale=1.0)
    r = cp.locate(g.GPD_BWD, Zb)
    assert r.outcome == CORRECTED and list(np.flatnonzero(cp.flags(r))) == [9]
    CT = cp.decode(g.GPD_BWD, Zb)
    assert op.rel_fro(CT, op.ref_backward(DT, W)) < REL_TOL
    # the oracle's own pipeline on the same inputs, seeds and nodes
    Ws_o = op.encode_W(W, code)
    for which, Z, Q, seed, mask, Zo in (
            (g.GPD_FWD, Zf, code.Q_f, 41, nodes_f, op.worker_products(Ws_o, op.encode_X(X, code))),
            (g.GPD_BWD, Zb, code.Q_b, 42, nodes_b, op.worker_products(op.encode_DeltaT(DT, code), Ws_o))):
        Zo = Zo.astype(np.float32)
        oinj.inject_gauss(Zo, seed, 1.0, nodes=[(mask >> p) & 1 for p in range(P)])
        ro = locate_subspace(Zo, code.points, Q, tolerances_for(np.float32))
        rg = cp.locate(which, Z)
        assert ro.outcome == rg.outcome and np.array_equal(ro.flagged, cp.flags(rg))
        got = S if which == g.GPD_FWD else CT
        assert op.rel_fro(got, op.decode(Zo, code, FWD if which == g.GPD_FWD else BWD, use=~ro.flagged)) < REL_TOL
    # coded update, then audit
    Dh, Xh = cp.encode(g.GPD_OPERAND_DELTA_UPD, Delta), cp.encode(g.GPD_OPERAND_X_UPD, X)
    g.gpd_update_shares(cp.plan, Wsh, Dh, Xh, c4.lr, 0.0)
    r = cp.locate(g.GPD_AUDIT, Wsh)
    assert r.outcome == NO_ERROR
    W_new = cp.decode(g.GPD_AUDIT, Wsh)
    ref_new = op.ref_update(W, Delta, X, c4.lr)
    assert op.rel_fro(W_new, ref_new) < REL_TOL
    assert op.rel_fro(W_new.astype(np.float64) - W, ref_new - W) < 5e-3
    assert g.gpd_device_status() == 0


# --------------------------------------------------------------------------------------------------
# config 3 at full size, in the launch configuration bench.py times: decisions against the oracle's
# (tests/golden/cfg3_full_expected.json, written by make_cfg3_expected.py from oracle/ alone),
# sampled worker outputs and sampled rows of the decoded product against FP64 definitions
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("precision", [g.GPD_PREC_AUTO, g.GPD_PREC_FP64_SLICED, g.GPD_PREC_FP64_SLICED40])
def test_config3_full_size_against_oracle_decisions(precision):
    import json
    import os
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "cfg3_full_expected.json")))
    cfg = wl.CONFIG_3_MATMUL
    assert gold["config"] == cfg.name
    W, X = wl.matmul_inputs(cfg)
    code = make_code(cfg)
    cp = CodedProduct(code, precision=precision)
    assert cp.np_dtype == np.float64
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    L = Z.numel() // cfg.P
    pos = np.array(gold["sample_positions"])
    got = host(Z.reshape(cfg.P, L)[:, torch.from_numpy(pos).cuda()])
    want = np.array(gold["clean_outputs_at_samples"])
    if precision in (g.GPD_PREC_FP64_SLICED, g.GPD_PREC_FP64_SLICED40):
        # digit planes: < 6e-15 (1.4e-12 with five planes) of (row scale x column scale) per term, sqrt(K) = 45
        # terms deep, scales within 4.07 x 4.5 standard deviations of each operand (bound derived in
        # test_gpu_sliced.py)
        assert np.abs(got - want).max() <= (3e-11 if precision == g.GPD_PREC_FP64_SLICED else 7e-9) * gold["scale"]
    else:
        assert np.abs(got - want).max() <= 1e-12 * gold["scale"] * 8      # FP64 products, K = 2048
    rows = np.arange(0, cfg.N1, cfg.N1 // 32)
    ref_rows = op.ref_forward(W[rows], X)
    for seed in cfg.inject_seeds:
        e = gold["seeds"][str(seed)]
        Zg = Z.clone()
        g.gpd_inject(cp.plan, g.GPD_FWD, Zg, seed, g.GPD_INJECT_ADDITIVE, prob=cfg.inject_prob, scale=gold["scale"])
        r = cp.locate(g.GPD_FWD, Zg)
        assert r.outcome == e["outcome"] and r.rank == e["rank"] and r.n_active == e["n_active"]
        assert list(np.flatnonzero(cp.flags(r))) == e["flagged"] == e["injected"]
        S = cp.decode(g.GPD_FWD, Zg)
        assert np.isfinite(S).all()
        assert op.rel_fro(S[rows], ref_rows) < REL_TOL
        # the decoded product must not depend on which nodes were hit: compare with the clean decode
        if seed == cfg.inject_seeds[0]:
            r0 = cp.locate(g.GPD_FWD, Z)
            assert r0.outcome == NO_ERROR
            S_clean = cp.decode(g.GPD_FWD, Z)
        assert op.rel_fro(S, S_clean) < REL_TOL


# --------------------------------------------------------------------------------------------------
# alternate substitution v = u^m, w = u^(mn): same kernels, other exponent tables
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N1,N0,B,m,n,d1,d2,P", [(384, 256, 64, 3, 2, 2, 2, 22), (512, 512, 64, 2, 2, 1, 1, 10)])
def test_alternate_substitution_products(N1, N0, B, m, n, d1, d2, P):
    from oracle.code import SUBST_V_UM
    code = GPCode(N1, N0, B, m, n, d1, d2, P, subst=SUBST_V_UM)
    assert P >= max(code.Q_f, code.Q_b) + 2
    cp = CodedProduct(code)
    W = (rand((N1, N0), 51) / np.sqrt(N0)).astype(np.float32)
    X, DT = rand((N0, B), 52), rand((B, N1), 53)
    Wsh = cp.encode_W(W)
    assert np.allclose(host(Wsh).reshape(P, N1 // m, N0 // n), op.encode_W(W, code), rtol=0, atol=1e-6)
    for which, operand, src, Q, ref, Zo in (
            (g.GPD_FWD, g.GPD_OPERAND_X_FWD, X, code.Q_f, op.ref_forward(W, X),
             op.worker_products(op.encode_W(W, code), op.encode_X(X, code))),
            (g.GPD_BWD, g.GPD_OPERAND_DELTAT_BWD, DT, code.Q_b, op.ref_backward(DT, W),
             op.worker_products(op.encode_DeltaT(DT, code), op.encode_W(W, code)))):
        Z = cp.products(which, cp.encode(operand, src))
        nodes = np.zeros(P, dtype=bool)
        nodes[[2]] = True
        g.gpd_inject(cp.plan, which, Z, 61, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=1 << 2, scale=1.0)
        Zo = Zo.astype(cp.np_dtype)
        oinj.inject_gauss(Zo, 61, 1.0, nodes=nodes)
        ro = locate_subspace(Zo, code.points, Q, tolerances_for(cp.np_dtype))
        r = cp.locate(which, Z)
        assert r.outcome == ro.outcome == CORRECTED and np.array_equal(cp.flags(r), ro.flagged)
        out = cp.decode(which, Z)
        assert op.rel_fro(out, ref) < REL_TOL
        assert op.rel_fro(out, op.decode(Zo, code, FWD if which == g.GPD_FWD else BWD, use=~ro.flagged)) < REL_TOL
    Delta = np.ascontiguousarray(DT.T)
    g.gpd_update_shares(cp.plan, Wsh, cp.encode(g.GPD_OPERAND_DELTA_UPD, Delta), cp.encode(g.GPD_OPERAND_X_UPD, X),
                        0.05, 0.0)
    assert cp.locate(g.GPD_AUDIT, Wsh).outcome == NO_ERROR
    assert op.rel_fro(cp.decode(g.GPD_AUDIT, Wsh), op.ref_update(W, Delta, X, 0.05)) < REL_TOL


# --------------------------------------------------------------------------------------------------
# limits and degenerate shapes
# --------------------------------------------------------------------------------------------------
def test_maximum_nodes_threshold_and_parity():
    """P = 64 nodes, threshold 32, 32 parity checks: the largest code a plan accepts."""
    N1, N0, B, m, n, d1 = 160, 96, 32, 5, 3, 2                        # Q_f = 5*3*2 + 3 - 1 = 32
    code = GPCode(N1, N0, B, m, n, d1, 1, 64)
    assert code.Q_f == 32
    cp = CodedProduct(code)
    assert cp.np_dtype == np.float64
    W, X = rand((N1, N0), 71), rand((N0, B), 72)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    r = cp.locate(g.GPD_FWD, Z)
    assert r.outcome == NO_ERROR
    nodes = np.zeros(64, dtype=bool)
    nodes[[4, 33, 60]] = True
    mask = sum(1 << int(p) for p in np.flatnonzero(nodes))
    g.gpd_inject(cp.plan, g.GPD_FWD, Z, 73, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=mask, scale=1.0)
    Zo = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    oinj.inject_gauss(Zo, 73, 1.0, nodes=nodes)
    ro = locate_subspace(Zo, code.points, code.Q_f, tolerances_for(np.float64))
    r = cp.locate(g.GPD_FWD, Z)
    assert r.outcome == ro.outcome == CORRECTED and np.array_equal(cp.flags(r), ro.flagged)
    assert np.array_equal(ro.flagged, nodes)
    # threshold 32 amplifies rounding by about 1e10 (the oracle itself reaches 5e-6 here)
    S = cp.decode(g.GPD_FWD, Z)
    assert op.rel_fro(S, op.decode(Zo, code, FWD, use=~ro.flagged)) < REL_TOL
    assert op.rel_fro(S, op.ref_forward(W, X)) < REL_TOL


def test_tiny_and_skinny_shapes():
    """One-element blocks, a single output position per node, and a mini-batch of one in the
    backward product (a 1 x K by K x N worker product)."""
    code = GPCode(2, 2, 1, 2, 2, 1, 1, 9)                            # blocks are 1 x 1, L = 1
    cp = CodedProduct(code, g.GPD_PREC_FP64)
    W, X, DT = rand((2, 2), 81), rand((2, 1), 82), rand((1, 2), 83)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    assert cp.locate(g.GPD_FWD, Z).outcome == NO_ERROR
    assert np.allclose(cp.decode(g.GPD_FWD, Z), W.astype(np.float64) @ X, atol=1e-6)
    Zb = cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT))
    assert np.allclose(cp.decode(g.GPD_BWD, Zb, use_mask=[True] * 9), DT.astype(np.float64) @ W, atol=1e-6)
    # one corrupted node with a single codeword: located (rank 1, one column of H in its range)
    Zg = Z.clone()
    Zg[5] += 3.0
    r = cp.locate(g.GPD_FWD, Zg)
    assert r.outcome == CORRECTED and list(np.flatnonzero(cp.flags(r))) == [5]
    # mini-batch of one, backward, FP32 path (thresholds 5 / 6): M = 1
    code = GPCode(256, 512, 1, 2, 2, 1, 1, 10)
    cp = CodedProduct(code)
    assert cp.np_dtype == np.float32
    W, DT = (rand((256, 512), 84) / 16).astype(np.float32), rand((1, 256), 85)
    cp.encode_W(W)
    Zb = cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT))
    assert cp.locate(g.GPD_BWD, Zb).outcome == NO_ERROR
    assert op.rel_fro(cp.decode(g.GPD_BWD, Zb), op.ref_backward(DT, W)) < REL_TOL


def test_bounded_wait_reports_timeout_and_leaves_the_context_usable():
    """A barrier wait that nothing ever satisfies gives up after its cycle limit: the status word reads
    GPD_ERR_TIMEOUT once, is cleared by the read, and later work runs normally."""
    assert g.gpd_device_status() == 0
    g.gpd_selftest_bounded_wait(100000)
    assert g.gpd_device_status() == g.GPD_ERR_TIMEOUT
    assert g.gpd_device_status() == 0
    code = GPCode(512, 512, 256, 2, 2, 1, 1, 10)
    cp = CodedProduct(code)
    W, X = rand((512, 512), 95), rand((512, 256), 96)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))      # tensor-core path, bounded waits inside
    assert cp.locate(g.GPD_FWD, Z).outcome == NO_ERROR
    assert op.rel_fro(cp.decode(g.GPD_FWD, Z), op.ref_forward(W, X)) < REL_TOL
    assert g.gpd_device_status() == 0


def test_plan_upload_and_forward_only_plan():
    plan = g.gpd_plan((96, 60, 6), (3, 2, 2, 3), 20)                    # Q_f = 13 <= 20 < Q_b = 22
    assert plan.query(g.GPD_Q_TABLES_ON_DEVICE) == 0
    g.gpd_plan_upload(plan)
    assert plan.query(g.GPD_Q_TABLES_ON_DEVICE) == 1
    g.gpd_plan_upload(plan)                                            # idempotent
    # a layer step that asks for the backward product is refused before anything is enqueued
    Wsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS).zero_()
    X = torch.zeros((60, 6), device="cuda")
    DT = torch.zeros((6, 96), device="cuda")
    S = torch.full((96, 6), 5.0, device="cuda")
    CT = torch.zeros((6, 60), device="cuda")
    with pytest.raises(g.GpdError) as e:
        g.coded_layer_step(plan, g.GPD_PHASE_FWD | g.GPD_PHASE_BWD, Wsh, X=X, DeltaT=DT, S_out=S, CT_out=CT,
                           results=g.new_results(3), workspace=plan.workspace(step=True))
    assert e.value.status == g.GPD_ERR_P_TOO_SMALL
    torch.cuda.synchronize()
    assert (S == 5.0).all()                                            # the forward phase did not run
