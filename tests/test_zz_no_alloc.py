"""gpd_locate_errors_static: error location for callers that may not allocate device memory.

Some users of this library run inside a job whose framework has already taken all of the GPU's
memory for its own pool, or in a loop where the device-wide stall of an allocation is not
acceptable.  For them the library offers one entry point whose scratch space is a fixed array
compiled into the library.  This test calls it through the C ABI, twice in a row (the array
keeps the previous call's contents and must be cleared by the call itself), on a plan that has
never been used by any other call, and checks every field of its result against the regular
gpd_locate_errors, the decision (outcome and flag vector) against the CPU oracle as well, and
that the plan it ran on still owns no device memory afterwards.  It is collected last so that a
run stopping at the first failure has already been through all other tests.
"""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import paper_1811_10751_b200 as g            # noqa: E402
from oracle import inject as oinj            # noqa: E402
from oracle.code import GPCode, powers       # noqa: E402
from oracle.locate import locate_subspace, tolerances_for   # noqa: E402


def _codewords(code, Q, L, seed, dtype):
    rng = np.random.default_rng(seed)
    return (powers(code.points, Q) @ rng.standard_normal((Q, L))).astype(dtype)


def _fields(r, P):
    return (r.outcome, r.n_flagged, r.rank, r.device_status, r.n_active,
            tuple(r.flagged[:P]), tuple(r.forced[:P]))


@pytest.mark.parametrize("prec,dtype", [(g.GPD_PREC_FP64, np.float64), (g.GPD_PREC_FP32, np.float32)])
def test_static_scratch_variant_matches_regular_entry_point_twice_in_a_row(prec, dtype):
    N1, N0, B, m, n, d, P = 256, 128, 64, 2, 2, 2, 15            # Q_f = 9, P - Q = 6
    code = GPCode(N1, N0, B, m, n, d, 1, P)
    L = (N1 // m) * (B // d)
    res_static, res_regular = g.new_results(1), g.new_results(1)
    cases = [
        (_codewords(code, code.Q_f, L, 1, dtype), None, (1 << 3) | (1 << 11)),      # two erroneous nodes
        (_codewords(code, code.Q_f, L, 2, dtype), None, 0),                          # clean: no error
        (_codewords(code, code.Q_f, L, 3, dtype), [p == 5 for p in range(P)], 1 << 9),   # erasure + error
        (_codewords(code, code.Q_f, L, 4, dtype), None, 0b111111),                   # six nodes: failure
    ]
    # the static entry point goes first, on a plan nothing else has touched
    plan_static = g.gpd_plan((N1, N0, B), (m, n, d, 1), P, precision=prec)
    plan_regular = g.gpd_plan((N1, N0, B), (m, n, d, 1), P, precision=prec)
    ws = plan_regular.workspace()
    outcomes = []
    for Z0, erased, mask in cases:
        Z = torch.from_numpy(Z0).cuda().reshape(-1)
        if mask:
            g.gpd_inject(plan_regular, g.GPD_FWD, Z, 77, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=mask, scale=1.0)
        # the oracle's decision on its own copy of the same seeded data
        Zr = Z0.copy()
        if mask:
            oinj.inject_gauss(Zr, 77, 1.0, nodes=[(mask >> p) & 1 == 1 for p in range(P)])
        ro = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(dtype), erased=erased)
        for _ in range(2):                                         # two calls in a row
            g.gpd_locate_errors_static(plan_static, g.GPD_FWD, Z, res_static, erased=erased)
            a = g.read_results(res_static)[0]
            g.gpd_locate_errors(plan_regular, g.GPD_FWD, Z, res_regular, ws, erased=erased)
            b = g.read_results(res_regular)[0]
            assert _fields(a, P) == _fields(b, P)
            assert a.outcome == ro.outcome and np.array_equal(np.array(a.flagged[:P], dtype=bool), ro.flagged)
            # nothing on the static path uploads the plan's tables (the library's only device allocation)
            assert plan_static.query(g.GPD_Q_TABLES_ON_DEVICE) == 0
            assert plan_regular.query(g.GPD_Q_TABLES_ON_DEVICE) == 1
            for x, y in ((a.residual, b.residual), (a.max_inside, b.max_inside), (a.min_outside, b.min_outside)):
                assert abs(x - y) <= 1e-9 * max(1.0, abs(y))
        outcomes.append(a.outcome)
    assert outcomes == [g.GPD_CORRECTED, g.GPD_NO_ERROR, g.GPD_CORRECTED, g.GPD_DECODE_FAILURE]


def test_static_scratch_variant_rejects_products_beyond_its_limit():
    # 4 x 4 split, P = 36: the audit product has P - Q = 20 parity checks, more than the built-in
    # scratch holds (16); the forward product (P - Q = 17) is over the limit too.
    plan = g.gpd_plan((256, 256, 32), (4, 4, 1, 1), 36)
    Z = plan.empty(g.GPD_Q_W_SHARE_ELEMS).zero_()
    res = g.new_results(1)
    for which in (g.GPD_AUDIT, g.GPD_FWD):
        with pytest.raises(g.GpdError) as e:
            g.gpd_locate_errors_static(plan, which, Z, res)
        assert e.value.status == g.GPD_ERR_STATIC_LIMIT
        assert "GPD_STATIC_MAX_PARITY" in str(e.value)
    # the backward product of the same plan (P - Q = 8) fits
    Zb = plan.empty(g.GPD_Q_OUT_ELEMS_BWD).zero_()
    g.gpd_locate_errors_static(plan, g.GPD_BWD, Zb, res)
    assert g.read_results(res)[0].outcome == g.GPD_NO_ERROR
