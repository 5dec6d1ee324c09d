"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its host
logic (plan construction, thresholds, tables, error codes) agrees with the oracle."""

import ctypes
import os
import re

import numpy as np
import pytest

import paper_1811_10751_b200 as g
from oracle.code import GPCode, chebyshev_points, parity_check, powers
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gpd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:gpd_status|const char\*)\s+(\w+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported():
    names = _declared_functions()
    assert "coded_layer_step" in names and "gpd_plan" in names and len(names) >= 18
    for n in names:
        assert hasattr(g.lib, n), f"{n} declared in include/gpd.h but not exported"
    assert sorted(g.EXPORTED) == names


def test_result_struct_layout_matches_header():
    # int32 x4, int64, double x3, 2 x 64 bytes
    assert g.RESULT_BYTES == 16 + 8 + 24 + 128
    assert g.gpd_locate_result.flagged.offset == 48 and g.gpd_locate_result.forced.offset == 112


def test_position_result_layout_workspace_query_and_argument_checks():
    import ctypes as C
    # int32 x4, int64 x4, 64 bytes
    assert g.POSITION_RESULT_BYTES == 16 + 32 + 64 and g.gpd_position_result.touched.offset == 48
    c = wl.CONFIG_3_MATMUL
    plan = g.gpd_plan((c.N1, c.N0, c.B), (c.m, c.n, c.d, 1), c.P)
    L = (c.N1 // c.m) * max(c.B // c.d, c.N0 // c.n)             # largest product of the plan (audit: N1/m x N0/n)
    # counters, the list of failing positions, and R + 1 doubles (syndrome, squared norm) for one position
    # in 32 of the product that needs most: here the audit product, R = P - Q_w = 17
    assert plan.query(g.GPD_Q_POSITION_WORKSPACE_BYTES) == 256 + 4 * L + (L // 32) * (17 + 1) * 8
    one = C.c_void_p(4096)                                        # never dereferenced: the checks come first
    assert g.lib.gpd_correct_positions(plan.handle, g.GPD_FWD, one, one, None, None) == g.GPD_ERR_WORKSPACE
    assert g.lib.gpd_correct_positions(plan.handle, g.GPD_FWD, None, one, one, None) == g.GPD_ERR_ARG
    assert g.lib.gpd_correct_positions(None, g.GPD_FWD, one, one, one, None) == g.GPD_ERR_ARG
    plan.destroy()


@pytest.mark.parametrize("shape,split,P", [
    ((64, 64, 64), (2, 2, 2, 1), 11), ((4096, 4096, 1), (4, 2, 1, 1), 13),
    ((8192, 8192, 512), (2, 4, 2, 1), 25), ((4096, 4096, 256), (2, 2, 1, 1), 10),
    ((8192, 1024, 1024), (4, 4, 1, 1), 36), ((10, 4096, 256), (2, 2, 1, 1), 10)])
def test_plan_thresholds_and_tables_match_oracle(shape, split, P):
    plan = g.gpd_plan(shape, split, P)
    code = GPCode(shape[0], shape[1], shape[2], split[0], split[1], split[2], split[3], P)
    assert plan.query(g.GPD_Q_THRESHOLD_FWD) == code.Q_f
    assert plan.query(g.GPD_Q_THRESHOLD_BWD) == code.Q_b
    assert plan.query(g.GPD_Q_THRESHOLD_AUDIT) == code.Q_w
    assert plan.query(g.GPD_Q_NODES) == P
    pts = plan.table(g.GPD_TABLE_POINTS)
    assert np.abs(pts - chebyshev_points(P)).max() < 1e-15
    pw = powers(pts, 64)
    assert np.allclose(plan.table(g.GPD_TABLE_COEF_W).reshape(P, -1),
                       pw[:, code.exp_W().reshape(-1)], rtol=1e-14, atol=0)
    assert np.allclose(plan.table(g.GPD_TABLE_COEF_X).reshape(P, -1),
                       pw[:, code.exp_X().reshape(-1)], rtol=1e-14, atol=0)
    assert np.allclose(plan.table(g.GPD_TABLE_COEF_DT).reshape(P, -1),
                       pw[:, code.exp_DeltaT().reshape(-1)], rtol=1e-14, atol=0)
    for tab, Q in ((g.GPD_TABLE_PARITY_FWD, code.Q_f), (g.GPD_TABLE_PARITY_AUDIT, code.Q_w)):
        H = plan.table(tab).reshape(P - Q, P)
        assert np.abs(H @ powers(pts, Q)).max() < 1e-13                  # H G^T = 0
        assert np.allclose(H @ H.T, np.eye(P - Q), atol=1e-13)
        Ho = parity_check(pts, Q)                                        # same row space as the oracle's
        assert np.abs(H - (H @ Ho.T) @ Ho).max() < 1e-6
    # precision rule: FP32 up to threshold 9, FP64 beyond
    qmax = max(code.Q_f, code.Q_b) if P >= code.Q_b else code.Q_f
    assert plan.query(g.GPD_Q_PRECISION) == (g.GPD_PREC_FP32 if qmax <= 9 else g.GPD_PREC_FP64)
    assert plan.query(g.GPD_Q_ELEMENT_SIZE) == (4 if qmax <= 9 else 8)
    N1, N0, B = shape
    m, n, d1, d2 = split
    assert plan.query(g.GPD_Q_W_SHARE_ELEMS) == P * (N1 // m) * (N0 // n)
    assert plan.query(g.GPD_Q_OUT_ELEMS_FWD) == P * (N1 // m) * (B // d1)
    plan.destroy()


def test_workload_configs_build_plans():
    for c in (wl.CONFIG_1_TINY, wl.CONFIG_2_MATVEC, wl.CONFIG_3_MATMUL):
        g.gpd_plan((c.N1, c.N0, c.B), (c.m, c.n, c.d, 1), c.P).destroy()


def test_plan_error_codes():
    def status(*a, **k):
        with pytest.raises(g.GpdError) as e:
            g.gpd_plan(*a, **k)
        return e.value.status
    assert status((10, 8, 4), (3, 2, 1, 1), 9) == g.GPD_ERR_SHAPE              # m does not divide N1
    assert status((8, 9, 4), (2, 2, 1, 1), 9) == g.GPD_ERR_SHAPE               # n does not divide N0
    assert status((8, 8, 5), (2, 2, 2, 1), 12) == g.GPD_ERR_SHAPE              # d1 does not divide B
    assert status((8, 8, 4), (2, 2, 1, 1), 4) == g.GPD_ERR_P_TOO_SMALL         # P < mn + n - 1 = 5
    assert status((64, 64, 64), (4, 4, 2, 1), 40) == g.GPD_ERR_Q_TOO_LARGE     # threshold 35 > 32
    assert status((8, 8, 4), (2, 2, 1, 1), 65) == g.GPD_ERR_Q_TOO_LARGE        # P > 64
    assert status((8, 8, 4), (2, 2, 1, 1), 6, points=[0, 1, 2, 3, 4, 4]) == g.GPD_ERR_POINTS
    assert status((8, 8, 4), (2, 2, 1, 1), 6, points=[0, 1, 2, 3, 4, np.nan]) == g.GPD_ERR_POINTS
    assert status((8, 8, 4), (2, 2, 1, 1), 6, precision=7) == g.GPD_ERR_ARG
    assert g.gpd_status_string(g.GPD_ERR_P_TOO_SMALL) == "fewer nodes than the recovery threshold"


def test_sliced_precision_plans():
    """Digit-plane storage: accepted when N0/n is a multiple of 16 and the block counts are ones the
    encoder is built for; element size and buffer sizes are those of the FP64 plan it stands in for."""
    c = wl.CONFIG_3_MATMUL
    plan = g.gpd_plan((c.N1, c.N0, c.B), (c.m, c.n, c.d, 1), c.P, precision=g.GPD_PREC_FP64_SLICED)
    ref = g.gpd_plan((c.N1, c.N0, c.B), (c.m, c.n, c.d, 1), c.P, precision=g.GPD_PREC_FP64)
    assert plan.query(g.GPD_Q_PRECISION) == g.GPD_PREC_FP64_SLICED and plan.query(g.GPD_Q_ELEMENT_SIZE) == 8
    for q in (g.GPD_Q_W_SHARE_ELEMS, g.GPD_Q_X_SHARE_ELEMS, g.GPD_Q_OUT_ELEMS_FWD, g.GPD_Q_THRESHOLD_FWD,
              g.GPD_Q_STEP_WORKSPACE_BYTES):
        assert plan.query(q) == ref.query(q)
    plan.destroy(), ref.destroy()
    for shape, split, P in (((64, 72, 8), (2, 2, 1, 1), 9),          # N0/n = 36
                            ((64, 160, 8), (2, 5, 1, 1), 20),        # 10 blocks per share of W
                            ((4, 32, 2), (1, 1, 1, 1), 2)):          # digit planes + scales would not fit
        with pytest.raises(g.GpdError) as e:
            g.gpd_plan(shape, split, P, precision=g.GPD_PREC_FP64_SLICED)
        assert e.value.status == g.GPD_ERR_UNSUPPORTED
    with pytest.raises(g.GpdError) as e:                              # coefficients up to 7e35: beyond the FP32 scale pass
        g.gpd_plan((64, 64, 8), (2, 2, 1, 1), 9, points=np.linspace(1e11, 9e11, 9), precision=g.GPD_PREC_FP64_SLICED)
    assert e.value.status == g.GPD_ERR_UNSUPPORTED


def test_custom_points_are_kept():
    pts = np.linspace(-0.9, 0.9, 7)
    plan = g.gpd_plan((8, 8, 4), (2, 2, 1, 1), 7, points=pts)
    assert np.array_equal(plan.table(g.GPD_TABLE_POINTS), pts)
    plan.destroy()


@pytest.mark.parametrize("shape,split,P", [((12, 8, 6), (3, 2, 2, 3), 26), ((4096, 4096, 256), (2, 2, 1, 1), 10),
                                           ((8192, 1024, 1024), (4, 4, 1, 1), 36)])
def test_alternate_substitution_plan_matches_oracle(shape, split, P):
    from oracle.code import SUBST_V_UM
    plan = g.gpd_plan_subst(shape, split, g.GPD_SUBST_V_EQ_UM, P)
    code = GPCode(shape[0], shape[1], shape[2], split[0], split[1], split[2], split[3], P, subst=SUBST_V_UM)
    assert plan.query(g.GPD_Q_THRESHOLD_FWD) == code.Q_f
    assert plan.query(g.GPD_Q_THRESHOLD_BWD) == code.Q_b
    assert plan.query(g.GPD_Q_THRESHOLD_AUDIT) == code.Q_w
    pw = powers(plan.table(g.GPD_TABLE_POINTS), 64)
    for tab, ex in ((g.GPD_TABLE_COEF_W, code.exp_W()), (g.GPD_TABLE_COEF_X, code.exp_X()),
                    (g.GPD_TABLE_COEF_DT, code.exp_DeltaT())):
        assert np.allclose(plan.table(tab).reshape(P, -1), pw[:, ex.reshape(-1)], rtol=1e-14, atol=0)
    H = plan.table(g.GPD_TABLE_PARITY_BWD).reshape(P - code.Q_b, P)
    assert np.abs(H @ powers(plan.table(g.GPD_TABLE_POINTS), code.Q_b)).max() < 1e-13
    plan.destroy()
    with pytest.raises(g.GpdError):
        g.gpd_plan_subst(shape, split, 7, P)
