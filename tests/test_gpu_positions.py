"""GPU parity of gpd_correct_positions (per-codeword correction under the adversarial model)
against the oracle: which positions are active / repaired / given up and which nodes are touched
must match exactly; repaired outputs and the decoded product within the floating-point bars."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import paper_1811_10751_b200 as g                        # noqa: E402
from oracle import product as op                         # noqa: E402
from oracle.code import GPCode, FWD, BWD                 # noqa: E402
from oracle.locate import (CORRECTED, DECODE_FAILURE, NO_ERROR, locate_subspace, tolerances_for)   # noqa: E402
from oracle.perpos import correct_positions              # noqa: E402
from tests.gpu_pipeline import CodedProduct, dev, host   # noqa: E402


def _scatter_errors(Z, t_max, frac, seed, scale):
    """Up to t_max errors per position on a random fraction of the positions; supports differ from
    position to position.  Z: [P, L] modified in place; returns the number of errors per position."""
    rng = np.random.default_rng(seed)
    P, L = Z.shape
    sizes = np.zeros(L, dtype=np.int64)
    hit = rng.random(L) < frac
    sizes[hit] = rng.integers(1, t_max + 1, size=int(hit.sum()))
    for l in np.flatnonzero(hit):
        nodes = rng.choice(P, size=sizes[l], replace=False)
        Z[nodes, l] += rng.choice([-1.0, 1.0], size=sizes[l]) * rng.uniform(0.25, 8.0, size=sizes[l]) * scale
    return sizes


@pytest.mark.parametrize("N1,N0,B,m,n,d1,P,prec", [
    (256, 256, 64, 2, 2, 2, 15, g.GPD_PREC_FP64),            # Q = 9,  R = 6, t = 3
    (256, 256, 64, 2, 2, 1, 9, g.GPD_PREC_FP32),             # Q = 5,  R = 4, t = 2, FP32 outputs
    (512, 512, 128, 2, 4, 2, 25, g.GPD_PREC_FP64_SLICED),    # Q = 19, R = 6, t = 3, digit-plane products
    (128, 128, 32, 2, 2, 1, 6, g.GPD_PREC_FP32),             # R = 1: nothing correctable, errors only detected
    (128, 128, 32, 2, 2, 2, 20, g.GPD_PREC_FP64),            # Q = 9,  R = 11, t = 5: the general (not unrolled) form
])
def test_positions_repaired_like_the_oracle(N1, N0, B, m, n, d1, P, prec):
    _check_against_oracle(N1, N0, B, m, n, d1, P, prec, frac=0.05)


def test_positions_more_failures_than_kept_syndromes():
    """The scan keeps the syndromes of the first 4096 failing positions for the repair (16384 positions
    here); with 40 % of the positions hit the repair reads the other codewords a second time.  Both routes
    must decide like the oracle."""
    _check_against_oracle(512, 512, 128, 2, 4, 2, 25, g.GPD_PREC_FP64, frac=0.4)


def _check_against_oracle(N1, N0, B, m, n, d1, P, prec, frac):
    rng = np.random.default_rng(N1 + P)
    W = (rng.standard_normal((N1, N0)) / np.sqrt(N0)).astype(np.float32)
    X = rng.standard_normal((N0, B)).astype(np.float32)
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    cp = CodedProduct(code, precision=prec)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    clean = cp.outputs_as_array(g.GPD_FWD, Z).reshape(P, -1).astype(np.float64)
    t = (P - code.Q_f) // 2
    scale = float(np.sqrt(np.mean(clean ** 2)))
    bad = clean.copy()
    sizes = _scatter_errors(bad, max(t, 1), frac, seed=7, scale=scale)
    Zg = dev(bad.astype(cp.np_dtype).reshape(-1))
    tol = tolerances_for(cp.np_dtype)
    ro = correct_positions(bad.astype(cp.np_dtype), code.points, code.Q_f, tol)
    r = g.gpd_correct_positions(cp.plan, g.GPD_FWD, Zg)
    assert (r.outcome, r.n_active, r.n_corrected, r.n_failed, r.n_entries, r.max_errors) == \
           (ro.outcome, ro.n_active, ro.n_corrected, ro.n_failed, ro.n_entries, ro.max_errors)
    assert np.array_equal(np.array(list(r.touched)[:P], dtype=bool), ro.touched)
    got = host(Zg).reshape(P, -1).astype(np.float64)
    eps = 1e-4 if cp.np_dtype == np.float32 else 1e-9
    assert np.abs(got - ro.corrected).max() <= eps * scale
    if t >= 1:
        assert r.outcome == CORRECTED and r.n_active == int((sizes > 0).sum()) and r.n_entries == int(sizes.sum())
        assert np.array(list(r.touched)[:P], dtype=bool).all()          # every node is blamed somewhere ...
        g.gpd_locate_errors(cp.plan, g.GPD_FWD, dev(bad.astype(cp.np_dtype).reshape(-1)), cp.res, cp.ws)
        assert g.read_results(cp.res)[0].outcome == DECODE_FAILURE      # ... which the node-level decision cannot serve
        S = cp.decode(g.GPD_FWD, Zg, use_mask=[True] * P)
        assert op.rel_fro(S, op.ref_forward(W, X)) < 1e-4
    else:
        assert r.outcome == DECODE_FAILURE and r.n_corrected == 0 and r.n_failed == r.n_active > 0
        assert np.array_equal(got, bad.astype(cp.np_dtype).astype(np.float64))   # nothing changed


def test_positions_clean_too_many_and_nonfinite():
    N1, N0, B, m, n, d1, P = 128, 128, 64, 2, 2, 1, 12        # Q = 5, R = 7, t = 3
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((N1, N0)) / np.sqrt(N0)).astype(np.float32)
    X = rng.standard_normal((N0, B)).astype(np.float32)
    code = GPCode(N1, N0, B, m, n, d1, 1, P)
    cp = CodedProduct(code, precision=g.GPD_PREC_FP64)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    r = g.gpd_correct_positions(cp.plan, g.GPD_FWD, Z.clone())
    assert r.outcome == NO_ERROR and r.n_active == 0 and not any(r.touched)
    clean = cp.outputs_as_array(g.GPD_FWD, Z).reshape(P, -1).astype(np.float64)
    bad = clean.copy()
    bad[[0, 3, 5, 8], 7] += np.array([1.0, -2.0, 1.5, 3.0])   # four errors: one too many
    bad[[1, 2, 11], 20] += 3.0                                # three: correctable
    bad[4, 100] = np.inf
    Zg = dev(bad.reshape(-1))
    ro = correct_positions(bad, code.points, code.Q_f, tolerances_for(np.float64))
    r = g.gpd_correct_positions(cp.plan, g.GPD_FWD, Zg)
    assert (ro.outcome, ro.n_active, ro.n_corrected, ro.n_failed) == (DECODE_FAILURE, 3, 1, 2)
    assert (r.outcome, r.n_active, r.n_corrected, r.n_failed, r.n_entries, r.max_errors) == \
           (ro.outcome, ro.n_active, ro.n_corrected, ro.n_failed, ro.n_entries, ro.max_errors)
    got = host(Zg).reshape(P, -1)
    assert np.array_equal(got[:, 7], bad[:, 7]) and np.array_equal(got[:, 100], bad[:, 100])
    assert np.abs(got[:, 20] - clean[:, 20]).max() < 1e-9
    assert [p for p in range(P) if r.touched[p]] == [1, 2, 11]


def test_positions_backward_product():
    N1, N0, B, m, n, d2, P = 256, 128, 64, 2, 2, 2, 16        # Q_b = 10, R = 6, t = 3
    rng = np.random.default_rng(8)
    W = (rng.standard_normal((N1, N0)) / np.sqrt(N0)).astype(np.float32)
    DT = rng.standard_normal((B, N1)).astype(np.float32)
    code = GPCode(N1, N0, B, m, n, 1, d2, P)
    cp = CodedProduct(code, precision=g.GPD_PREC_FP64)
    cp.encode_W(W)
    Z = cp.products(g.GPD_BWD, cp.encode(g.GPD_OPERAND_DELTAT_BWD, DT))
    clean = cp.outputs_as_array(g.GPD_BWD, Z).reshape(P, -1).astype(np.float64)
    bad = clean.copy()
    sizes = _scatter_errors(bad, 3, 0.1, seed=2, scale=float(np.sqrt(np.mean(clean ** 2))))
    Zg = dev(bad.reshape(-1))
    ro = correct_positions(bad, code.points, code.Q_b, tolerances_for(np.float64))
    r = g.gpd_correct_positions(cp.plan, g.GPD_BWD, Zg)
    assert (r.outcome, r.n_active, r.n_entries) == (ro.outcome, ro.n_active, ro.n_entries) == \
           (CORRECTED, int((sizes > 0).sum()), int(sizes.sum()))
    CT = cp.decode(g.GPD_BWD, Zg, use_mask=[True] * P)
    assert op.rel_fro(CT, op.ref_backward(DT, W)) < 1e-4


def test_positions_full_size_outputs_on_a_sample():
    """The 8192 x 8192 x 512 product's outputs (P = 25, 1.05 M positions, digit-plane products) with
    1-3 errors on 1 % of the positions, in the launch configuration the benchmark times.  The oracle
    repairs a sample of 20 000 positions that holds every corrupted one; counters must match, and
    the sampled outputs must come back as the oracle leaves them."""
    import workloads as wl
    cfg = wl.CONFIG_3_MATMUL
    W, X = wl.matmul_inputs(cfg)
    code = GPCode(cfg.N1, cfg.N0, cfg.B, cfg.m, cfg.n, cfg.d, 1, cfg.P)
    cp = CodedProduct(code, precision=g.GPD_PREC_FP64_SLICED)
    cp.encode_W(W)
    Z = cp.products(g.GPD_FWD, cp.encode(g.GPD_OPERAND_X_FWD, X))
    P, L = cfg.P, Z.numel() // cfg.P
    rng = np.random.default_rng(99)
    sample = np.sort(rng.choice(L, size=20000, replace=False))
    hit = rng.choice(sample, size=L // 100, replace=False)
    sizes = rng.integers(1, 4, size=hit.size)
    pos = np.repeat(hit, sizes)
    node = np.concatenate([rng.choice(P, size=k, replace=False) for k in sizes])
    scale = float(Z.pow(2).mean().sqrt())
    val = rng.choice([-1.0, 1.0], size=pos.size) * rng.uniform(0.25, 8.0, size=pos.size) * scale
    Zv = Z.view(P, L)
    Zv[torch.from_numpy(node).cuda(), torch.from_numpy(pos).cuda()] += torch.from_numpy(val).cuda()
    smp = torch.from_numpy(sample).cuda()
    bad_sample = host(Zv[:, smp])
    ro = correct_positions(bad_sample, code.points, code.Q_f, tolerances_for(np.float64))
    r = g.gpd_correct_positions(cp.plan, g.GPD_FWD, Z)
    assert (r.outcome, r.n_active, r.n_corrected, r.n_failed, r.n_entries, r.max_errors) == \
           (ro.outcome, ro.n_active, ro.n_corrected, ro.n_failed, ro.n_entries, ro.max_errors) == \
           (CORRECTED, hit.size, hit.size, 0, int(sizes.sum()), 3)
    assert np.array_equal(np.array(list(r.touched)[:P], dtype=bool), ro.touched)
    assert np.abs(host(Zv[:, smp]) - ro.corrected).max() <= 1e-9 * scale
    rows = np.arange(0, cfg.N1, cfg.N1 // 32)
    S = cp.decode(g.GPD_FWD, Z, use_mask=[True] * P)
    assert op.rel_fro(S[rows], op.ref_forward(W[rows], X)) < 1e-4
