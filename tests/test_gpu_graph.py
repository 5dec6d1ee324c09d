"""The library's compute calls only enqueue work on the stream they are given, and a plan whose
tables were uploaded beforehand allocates nothing: a whole coded product (encode of X, node products,
injection, location, decode) can therefore be captured into a CUDA graph as it is.  The replayed graph
must leave exactly what the same calls leave when they run eagerly."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import os                                    # noqa: E402

if any(k in os.environ for k in ("CUDA_INJECTION64_PATH", "NV_COMPUTE_PROFILER_PERFWORKS_DIR", "NV_NSIGHT_INJECTION_PORT_BASE")):
    pytest.skip("a profiler is attached: ncu ends a process that launches into a stream capture", allow_module_level=True)

import paper_1811_10751_b200 as g            # noqa: E402


@pytest.mark.parametrize("shape,split,P,prec", [
    ((512, 512, 128), (2, 2, 2, 1), 15, g.GPD_PREC_FP64),            # FP64 mma products
    ((512, 512, 256), (2, 2, 1, 1), 10, g.GPD_PREC_FP32),            # tcgen05 3xTF32 products (TMA maps built per launch)
    ((512, 512, 128), (2, 4, 2, 1), 25, g.GPD_PREC_FP64_SLICED),     # int8 digit planes
])
def test_coded_product_replayed_from_a_cuda_graph_equals_the_eager_calls(shape, split, P, prec):
    N1, N0, B = shape
    gen = torch.Generator(device="cuda").manual_seed(N1 + P)
    W = torch.randn((N1, N0), device="cuda", generator=gen) / N0 ** 0.5
    X = torch.randn((N0, B), device="cuda", generator=gen)
    plan = g.gpd_plan(shape, split, P, precision=prec)
    g.gpd_plan_upload(plan)                                          # the one allocation, outside the capture
    Wsh, Xsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS), plan.empty(g.GPD_Q_X_SHARE_ELEMS)
    Z = plan.empty(g.GPD_Q_OUT_ELEMS_FWD)
    S = torch.empty((N1, B), dtype=torch.float32, device="cuda")
    ws, res = plan.workspace(), g.new_results(1)
    g.gpd_encode_A(plan, W, Wsh)
    stream = torch.cuda.Stream()

    def product(st):
        g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, X, Xsh, stream=st)
        g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z, stream=st)
        g.gpd_inject(plan, g.GPD_FWD, Z, 7, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=1 << 3, scale=1.0, stream=st)
        g.gpd_locate_errors(plan, g.GPD_FWD, Z, res, ws, stream=st)
        g.gpd_decode(plan, g.GPD_FWD, Z, S, ws, result=res, stream=st)

    with torch.cuda.stream(stream):
        product(stream)
    torch.cuda.synchronize()
    eager_S, eager_Z = S.clone(), Z.clone()
    eager_r = g.read_results(res)[0]
    eager_flags = list(eager_r.flagged)[:P]
    assert eager_r.outcome == g.GPD_CORRECTED and [p for p in range(P) if eager_flags[p]] == [3]

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        product(stream)
    for _ in range(2):
        S.fill_(float("nan"))
        Z.fill_(float("nan"))
        with torch.cuda.stream(stream):
            graph.replay()
        torch.cuda.synchronize()
        r = g.read_results(res)[0]
        assert (r.outcome, list(r.flagged)[:P]) == (eager_r.outcome, eager_flags)
        assert torch.equal(Z, eager_Z) and torch.equal(S, eager_S)
    assert g.gpd_device_status() == 0
    plan.destroy()


def test_encoding_update_audit_regeneration_and_position_repair_under_capture():
    """The remaining compute calls: initial encoding of W, the coded update, share-error injection, the audit
    with regeneration of the flagged share, and the per-position repair of a forward product."""
    N1, N0, B, P = 256, 256, 64, 15
    gen = torch.Generator(device="cuda").manual_seed(5)
    W = torch.randn((N1, N0), device="cuda", generator=gen) / N0 ** 0.5
    X = torch.randn((N0, B), device="cuda", generator=gen)
    D = torch.randn((N1, B), device="cuda", generator=gen) / B
    plan = g.gpd_plan((N1, N0, B), (2, 2, 2, 1), P, precision=g.GPD_PREC_FP64)       # Q_f = 9, Q_w = 4
    g.gpd_plan_upload(plan)
    Wsh, Xsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS), plan.empty(g.GPD_Q_X_SHARE_ELEMS)
    Dh, Xh = plan.empty(g.GPD_Q_DHAT_ELEMS), plan.empty(g.GPD_Q_XHAT_ELEMS)
    Z = plan.empty(g.GPD_Q_OUT_ELEMS_FWD)
    ws, res = plan.workspace(), g.new_results(1)
    ws_pos = torch.empty(plan.query(g.GPD_Q_POSITION_WORKSPACE_BYTES), dtype=torch.uint8, device="cuda")
    res_pos = torch.zeros(g.POSITION_RESULT_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    L = Z.numel() // P

    def work(st):
        g.gpd_encode_A(plan, W, Wsh, stream=st)
        g.gpd_encode_B(plan, g.GPD_OPERAND_DELTA_UPD, D, Dh, stream=st)
        g.gpd_encode_B(plan, g.GPD_OPERAND_X_UPD, X, Xh, stream=st)
        g.gpd_update_shares(plan, Wsh, Dh, Xh, 0.0625, 0.125, stream=st)
        g.gpd_inject(plan, g.GPD_AUDIT, Wsh, 11, g.GPD_INJECT_GAUSS, prob=-1.0, node_mask=1 << 6, scale=1.0, stream=st)
        g.gpd_locate_errors(plan, g.GPD_AUDIT, Wsh, res, ws, stream=st)
        g.gpd_regenerate_shares(plan, Wsh, res, ws, stream=st)
        g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, X, Xsh, stream=st)
        g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z, stream=st)
        g.gpd_inject(plan, g.GPD_FWD, Z, 3, g.GPD_INJECT_BITFLIP, count=2, scale=1.0, stream=st)
        g.gpd_correct_positions(plan, g.GPD_FWD, Z, workspace=ws_pos, result=res_pos, stream=st)

    with torch.cuda.stream(stream):
        work(stream)
    torch.cuda.synchronize()
    eager_W, eager_Z = Wsh.clone(), Z.clone()
    eager_audit = g.read_results(res)[0]
    eager_pos = g.read_position_result(res_pos)
    assert eager_audit.outcome == g.GPD_CORRECTED and [p for p in range(P) if eager_audit.flagged[p]] == [6]
    assert eager_pos.outcome == g.GPD_CORRECTED and eager_pos.n_corrected == 2

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        work(stream)
    Wsh.fill_(float("nan"))
    Z.fill_(float("nan"))
    with torch.cuda.stream(stream):
        graph.replay()
    torch.cuda.synchronize()
    audit, pos = g.read_results(res)[0], g.read_position_result(res_pos)
    assert (audit.outcome, list(audit.flagged)[:P]) == (eager_audit.outcome, list(eager_audit.flagged)[:P])
    assert (pos.outcome, pos.n_active, pos.n_corrected, pos.n_entries) == \
           (eager_pos.outcome, eager_pos.n_active, eager_pos.n_corrected, eager_pos.n_entries)
    assert torch.equal(Wsh, eager_W) and torch.equal(Z, eager_Z)
    assert g.gpd_device_status() == 0
    plan.destroy()
