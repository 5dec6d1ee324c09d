"""ctypes binding of libgpd.so: same names as the C ABI (include/gpd.h), argument marshalling only.

Every step of the coded product runs in the library's CUDA kernels; PyTorch is used here only
to own device memory and streams.  There is no CPU fallback: if the shared library is missing,
importing this module fails.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgpd.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} not found: build it with `python paper_1811_10751_b200/build.py` "
        "(nvcc, sm_100a). This package has no CPU fallback.")
lib = C.CDLL(_LIB_PATH)

# ---- enums ------------------------------------------------------------------------------------
GPD_OK = 0
(GPD_ERR_ARG, GPD_ERR_SHAPE, GPD_ERR_POINTS, GPD_ERR_P_TOO_SMALL, GPD_ERR_Q_TOO_LARGE,
 GPD_ERR_WORKSPACE, GPD_ERR_CUDA, GPD_ERR_TIMEOUT, GPD_ERR_UNSUPPORTED, GPD_ERR_STATIC_LIMIT) = range(1, 11)
GPD_NO_ERROR, GPD_CORRECTED, GPD_DECODE_FAILURE = 0, 1, 2
GPD_FWD, GPD_BWD, GPD_UPD, GPD_AUDIT = 0, 1, 2, 3
GPD_OPERAND_X_FWD, GPD_OPERAND_DELTAT_BWD, GPD_OPERAND_DELTA_UPD, GPD_OPERAND_X_UPD = 0, 1, 2, 3
GPD_PREC_AUTO, GPD_PREC_FP32, GPD_PREC_FP64, GPD_PREC_FP64_SLICED, GPD_PREC_FP64_SLICED40 = 0, 1, 2, 3, 4
GPD_PREC_FP64_SLICED_TRAIN = 5
GPD_INJECT_BITFLIP, GPD_INJECT_ADDITIVE, GPD_INJECT_GAUSS = 0, 1, 2
GPD_ACT_IDENTITY, GPD_ACT_RELU, GPD_ACT_SIGMOID = 0, 1, 2
GPD_PHASE_FWD, GPD_PHASE_BWD, GPD_PHASE_UPD, GPD_PHASE_REGEN, GPD_PHASE_INJECT_SHARES = 1, 2, 4, 8, 16
(GPD_Q_THRESHOLD_FWD, GPD_Q_THRESHOLD_BWD, GPD_Q_THRESHOLD_AUDIT, GPD_Q_ELEMENT_SIZE,
 GPD_Q_W_SHARE_ELEMS, GPD_Q_X_SHARE_ELEMS, GPD_Q_DT_SHARE_ELEMS, GPD_Q_DHAT_ELEMS, GPD_Q_XHAT_ELEMS,
 GPD_Q_OUT_ELEMS_FWD, GPD_Q_OUT_ELEMS_BWD, GPD_Q_WORKSPACE_BYTES, GPD_Q_STEP_WORKSPACE_BYTES,
 GPD_Q_PRECISION, GPD_Q_NODES, GPD_Q_POSITION_WORKSPACE_BYTES, GPD_Q_TABLES_ON_DEVICE) = range(17)
(GPD_TABLE_POINTS, GPD_TABLE_PARITY_FWD, GPD_TABLE_PARITY_BWD, GPD_TABLE_PARITY_AUDIT,
 GPD_TABLE_COEF_W, GPD_TABLE_COEF_X, GPD_TABLE_COEF_DT) = range(7)
GPD_MAX_NODES = 64
GPD_SUBST_U_EQ_VN, GPD_SUBST_V_EQ_UM = 0, 1

EXPORTED = [
    "gpd_status_string", "gpd_plan", "gpd_plan_subst", "gpd_plan_upload", "gpd_selftest_bounded_wait", "gpd_plan_destroy", "gpd_plan_query", "gpd_plan_table",
    "gpd_encode_A", "gpd_encode_B", "gpd_worker_gemm", "gpd_device_status", "gpd_update_shares", "gpd_inject",
    "gpd_locate_errors", "gpd_locate_errors_static", "gpd_correct_positions", "gpd_decode", "gpd_regenerate_shares", "gpd_activation", "gpd_softmax_xent_delta",
    "gpd_backprop_hadamard", "gpd_sae_output_delta", "gpd_sae_hidden_delta", "coded_layer_step",
]


class gpd_shape(C.Structure):
    _fields_ = [("N1", C.c_int64), ("N0", C.c_int64), ("B", C.c_int64)]


class gpd_split(C.Structure):
    _fields_ = [("m", C.c_int32), ("n", C.c_int32), ("d1", C.c_int32), ("d2", C.c_int32)]


class gpd_locate_result(C.Structure):
    _fields_ = [("outcome", C.c_int32), ("n_flagged", C.c_int32), ("rank", C.c_int32),
                ("device_status", C.c_int32), ("n_active", C.c_int64), ("residual", C.c_double),
                ("max_inside", C.c_double), ("min_outside", C.c_double),
                ("flagged", C.c_uint8 * GPD_MAX_NODES), ("forced", C.c_uint8 * GPD_MAX_NODES)]


RESULT_BYTES = C.sizeof(gpd_locate_result)


class gpd_position_result(C.Structure):
    _fields_ = [("outcome", C.c_int32), ("max_errors", C.c_int32), ("device_status", C.c_int32),
                ("reserved", C.c_int32), ("n_active", C.c_int64), ("n_corrected", C.c_int64),
                ("n_failed", C.c_int64), ("n_entries", C.c_int64), ("touched", C.c_uint8 * GPD_MAX_NODES)]


POSITION_RESULT_BYTES = C.sizeof(gpd_position_result)

_vp, _i32, _i64, _u64, _f, _d = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float, C.c_double
lib.gpd_status_string.restype = C.c_char_p
lib.gpd_status_string.argtypes = [C.c_int]
lib.gpd_plan.argtypes = [C.POINTER(gpd_shape), C.POINTER(gpd_split), _i32, C.POINTER(C.c_double), C.c_int,
                         C.POINTER(_vp)]
lib.gpd_plan_subst.argtypes = [C.POINTER(gpd_shape), C.POINTER(gpd_split), C.c_int, _i32, C.POINTER(C.c_double),
                               C.c_int, C.POINTER(_vp)]
lib.gpd_plan_destroy.argtypes = [_vp]
lib.gpd_plan_upload.argtypes = [_vp]
lib.gpd_selftest_bounded_wait.argtypes = [_i64, _vp]
lib.gpd_plan_query.argtypes = [_vp, C.c_int, C.POINTER(_i64)]
lib.gpd_plan_table.argtypes = [_vp, C.c_int, C.POINTER(C.c_double), _i64, C.POINTER(_i64)]
lib.gpd_encode_A.argtypes = [_vp, _vp, _vp, _vp]
lib.gpd_encode_B.argtypes = [_vp, C.c_int, _vp, _vp, _vp]
lib.gpd_worker_gemm.argtypes = [_vp, C.c_int, _vp, _vp, _vp, _vp]
lib.gpd_device_status.argtypes = [C.POINTER(_i32)]
lib.gpd_update_shares.argtypes = [_vp, _vp, _vp, _vp, _f, _f, _vp, _vp]
lib.gpd_inject.argtypes = [_vp, C.c_int, _vp, _u64, C.c_int, _d, _u64, _i32, _d, _vp, _vp]
lib.gpd_locate_errors.argtypes = [_vp, C.c_int, _vp, C.POINTER(C.c_uint8), _vp, _vp, _vp]
lib.gpd_locate_errors_static.argtypes = [_vp, C.c_int, _vp, C.POINTER(C.c_uint8), _vp, _vp]
lib.gpd_correct_positions.argtypes = [_vp, C.c_int, _vp, _vp, _vp, _vp]
lib.gpd_decode.argtypes = [_vp, C.c_int, _vp, C.POINTER(C.c_uint8), _vp, _vp, _vp, C.c_int, _vp, _vp]
lib.gpd_regenerate_shares.argtypes = [_vp, _vp, _vp, _vp, _vp]
lib.gpd_activation.argtypes = [C.c_int, _vp, _vp, _i64, _vp]
lib.gpd_softmax_xent_delta.argtypes = [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _vp]
lib.gpd_backprop_hadamard.argtypes = [C.c_int, _vp, _vp, _vp, _vp, _i64, _i64, _vp]
lib.gpd_sae_output_delta.argtypes = [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _vp]
lib.gpd_sae_hidden_delta.argtypes = [_vp, _vp, _f, _f, _vp, _vp, _vp, _i64, _i64, _vp]
lib.coded_layer_step.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp, C.c_int, _f, _f, _u64, _d, _d, _vp, _vp, _vp,
                                 _vp, _vp, _vp]
for _name in EXPORTED:
    if _name != "gpd_status_string":
        getattr(lib, _name).restype = C.c_int


class GpdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.gpd_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != GPD_OK:
        raise GpdError(status, where)


def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype] = None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensor expected")
    if not t.is_contiguous():
        raise ValueError("contiguous tensor expected")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"tensor of dtype {dtype} expected, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


_F32 = torch.float32


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _mask(mask: Optional[Sequence[bool]], P: int):
    if mask is None:
        return None
    arr = (C.c_uint8 * P)(*[1 if b else 0 for b in mask])
    return arr


class Plan:
    """Owner of a gpd_plan_t handle."""

    def __init__(self, handle: int, shape, split, P: int):
        self.handle = C.c_void_p(handle)
        self.shape, self.split, self.P = shape, split, P

    def query(self, what: int) -> int:
        v = _i64(0)
        _check(lib.gpd_plan_query(self.handle, what, C.byref(v)), "gpd_plan_query")
        return int(v.value)

    def table(self, which: int) -> np.ndarray:
        n = _i64(0)
        _check(lib.gpd_plan_table(self.handle, which, None, 0, C.byref(n)), "gpd_plan_table")
        out = np.empty(int(n.value), dtype=np.float64)
        if n.value:
            _check(lib.gpd_plan_table(self.handle, which, out.ctypes.data_as(C.POINTER(C.c_double)), n, C.byref(n)),
                   "gpd_plan_table")
        return out

    @property
    def dtype(self) -> torch.dtype:
        return torch.float32 if self.query(GPD_Q_ELEMENT_SIZE) == 4 else torch.float64

    def empty(self, what: int, device="cuda") -> torch.Tensor:
        """Uninitialised device buffer of the plan's storage type holding `what` elements."""
        return torch.empty(self.query(what), dtype=self.dtype, device=device)

    def workspace(self, step: bool = False, device="cuda") -> torch.Tensor:
        n = self.query(GPD_Q_STEP_WORKSPACE_BYTES if step else GPD_Q_WORKSPACE_BYTES)
        return torch.empty(n, dtype=torch.uint8, device=device)

    def destroy(self):
        if self.handle:
            lib.gpd_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def gpd_status_string(status: int) -> str:
    return lib.gpd_status_string(status).decode()


def gpd_plan(shape, split, P: int, points=None, precision: int = GPD_PREC_AUTO,
             subst: int = GPD_SUBST_U_EQ_VN) -> Plan:
    """shape = (N1, N0, B); split = (m, n, d1, d2); points: P doubles or None (Chebyshev);
    subst other than the default goes through gpd_plan_subst."""
    sh = gpd_shape(*[int(v) for v in shape])
    sp = gpd_split(*[int(v) for v in split])
    pts = None
    if points is not None:
        arr = np.ascontiguousarray(points, dtype=np.float64)
        if arr.size != P:
            raise ValueError("need exactly P points")
        pts = arr.ctypes.data_as(C.POINTER(C.c_double))
    h = _vp(0)
    if subst == GPD_SUBST_U_EQ_VN:
        _check(lib.gpd_plan(C.byref(sh), C.byref(sp), int(P), pts, int(precision), C.byref(h)), "gpd_plan")
    else:
        _check(lib.gpd_plan_subst(C.byref(sh), C.byref(sp), int(subst), int(P), pts, int(precision), C.byref(h)),
               "gpd_plan_subst")
    return Plan(h.value, tuple(shape), tuple(split), int(P))


def gpd_plan_subst(shape, split, subst: int, P: int, points=None, precision: int = GPD_PREC_AUTO) -> Plan:
    return gpd_plan(shape, split, P, points=points, precision=precision, subst=subst)


def gpd_plan_destroy(plan: Plan):
    plan.destroy()


def gpd_plan_upload(plan: Plan):
    """Uploads the plan's tables to the current device now instead of at the first compute call."""
    _check(lib.gpd_plan_upload(plan.handle), "gpd_plan_upload")


def gpd_selftest_bounded_wait(limit_cycles: int = 100000, stream=None):
    """Launches a one-CTA kernel whose barrier wait must run out; gpd_device_status() then reports
    GPD_ERR_TIMEOUT once."""
    _check(lib.gpd_selftest_bounded_wait(int(limit_cycles), _stream(stream)), "gpd_selftest_bounded_wait")


def gpd_encode_A(plan: Plan, W, W_shares, stream=None):
    _check(lib.gpd_encode_A(plan.handle, _ptr(W, _F32), _ptr(W_shares, plan.dtype), _stream(stream)), "gpd_encode_A")


def gpd_encode_B(plan: Plan, operand: int, src, shares, stream=None):
    _check(lib.gpd_encode_B(plan.handle, operand, _ptr(src, _F32), _ptr(shares, plan.dtype), _stream(stream)), "gpd_encode_B")


def gpd_worker_gemm(plan: Plan, which: int, W_shares, other_shares, outputs, stream=None):
    _check(lib.gpd_worker_gemm(plan.handle, which, _ptr(W_shares), _ptr(other_shares), _ptr(outputs),
                               _stream(stream)), "gpd_worker_gemm")


def gpd_device_status() -> int:
    """Synchronises the device and returns (then clears) the tensor-path status word."""
    v = _i32(0)
    _check(lib.gpd_device_status(C.byref(v)), "gpd_device_status")
    return int(v.value)


def gpd_update_shares(plan: Plan, W_shares, Dhat, Xhat, eta: float, lam: float = 0.0, gate=None, stream=None):
    _check(lib.gpd_update_shares(plan.handle, _ptr(W_shares), _ptr(Dhat), _ptr(Xhat), eta, lam, _ptr(gate),
                                 _stream(stream)), "gpd_update_shares")


def gpd_inject(plan: Plan, which: int, outputs, seed: int, mode: int, prob: float = -1.0, node_mask: int = 0,
               count: int = 0, scale: float = 1.0, hit_mask=None, stream=None):
    _check(lib.gpd_inject(plan.handle, which, _ptr(outputs), seed & 0xFFFFFFFFFFFFFFFF, mode, prob,
                          node_mask & 0xFFFFFFFFFFFFFFFF, count, scale, _ptr(hit_mask), _stream(stream)),
           "gpd_inject")


def gpd_locate_errors(plan: Plan, which: int, outputs, result, workspace, erased=None, stream=None):
    _check(lib.gpd_locate_errors(plan.handle, which, _ptr(outputs), _mask(erased, plan.P), _ptr(result),
                                 _ptr(workspace), _stream(stream)), "gpd_locate_errors")


def gpd_locate_errors_static(plan: Plan, which: int, outputs, result, erased=None, stream=None):
    """gpd_locate_errors without a workspace and without any device allocation on its path: the
    scratch is a fixed array inside the library (products with P - Q <= 16 only).  Calls on one GPU
    share that array, so keep them ordered on one stream."""
    _check(lib.gpd_locate_errors_static(plan.handle, which, _ptr(outputs), _mask(erased, plan.P), _ptr(result),
                                        _stream(stream)), "gpd_locate_errors_static")


def gpd_correct_positions(plan: Plan, which: int, outputs, workspace=None, result=None, stream=None):
    """Repairs every output position on its own (up to floor((P-Q)/2) errors each), in place.  With
    `result` (a device buffer of POSITION_RESULT_BYTES) the call only enqueues work; without it the
    result struct is copied back to the host and returned (synchronises)."""
    if workspace is None:
        workspace = torch.empty(plan.query(GPD_Q_POSITION_WORKSPACE_BYTES), dtype=torch.uint8, device=outputs.device)
    res = result if result is not None else torch.zeros(POSITION_RESULT_BYTES, dtype=torch.uint8, device=outputs.device)
    _check(lib.gpd_correct_positions(plan.handle, which, _ptr(outputs, plan.dtype), _ptr(res), _ptr(workspace),
                                     _stream(stream)), "gpd_correct_positions")
    return None if result is not None else read_position_result(res)


def read_position_result(buf: torch.Tensor) -> gpd_position_result:
    return gpd_position_result.from_buffer_copy(buf.cpu().numpy().tobytes())


def gpd_decode(plan: Plan, which: int, outputs, out, workspace, result=None, use_mask=None, act_out=None,
               activation: int = GPD_ACT_IDENTITY, stream=None):
    _check(lib.gpd_decode(plan.handle, which, _ptr(outputs), _mask(use_mask, plan.P), _ptr(result), _ptr(out, _F32),
                          _ptr(act_out, _F32), activation, _ptr(workspace), _stream(stream)), "gpd_decode")


def gpd_regenerate_shares(plan: Plan, W_shares, result, workspace, stream=None):
    _check(lib.gpd_regenerate_shares(plan.handle, _ptr(W_shares, plan.dtype), _ptr(result), _ptr(workspace),
                                     _stream(stream)), "gpd_regenerate_shares")


def gpd_activation(kind: int, S, X_next, stream=None):
    _check(lib.gpd_activation(kind, _ptr(S), _ptr(X_next), S.numel(), _stream(stream)), "gpd_activation")


def gpd_softmax_xent_delta(S, labels, Delta, DeltaT, loss, stream=None):
    Cn, B = S.shape
    _check(lib.gpd_softmax_xent_delta(_ptr(S), _ptr(labels), _ptr(Delta), _ptr(DeltaT), _ptr(loss), Cn, B,
                                      _stream(stream)), "gpd_softmax_xent_delta")


def gpd_backprop_hadamard(kind: int, CT, X, Delta, DeltaT, stream=None):
    N, B = X.shape
    _check(lib.gpd_backprop_hadamard(kind, _ptr(CT), _ptr(X), _ptr(Delta), _ptr(DeltaT), N, B, _stream(stream)),
           "gpd_backprop_hadamard")


def gpd_sae_output_delta(S2, X, Delta2, Delta2T, loss, stream=None):
    N, B = X.shape
    _check(lib.gpd_sae_output_delta(_ptr(S2), _ptr(X), _ptr(Delta2), _ptr(Delta2T), _ptr(loss), N, B,
                                    _stream(stream)), "gpd_sae_output_delta")


def gpd_sae_hidden_delta(C2T, Y1, rho: float, beta: float, Delta1, Delta1T, kl_loss, stream=None):
    N, B = Y1.shape
    _check(lib.gpd_sae_hidden_delta(_ptr(C2T), _ptr(Y1), rho, beta, _ptr(Delta1), _ptr(Delta1T), _ptr(kl_loss),
                                    N, B, _stream(stream)), "gpd_sae_hidden_delta")


def coded_layer_step(plan: Plan, phases: int, W_shares, X=None, Delta=None, DeltaT=None,
                     activation: int = GPD_ACT_IDENTITY, eta: float = 0.0, lam: float = 0.0,
                     inject_seed: int = 0, inject_prob: float = 0.0, inject_scale: float = 1.0,
                     S_out=None, Xnext_out=None, CT_out=None, results=None, workspace=None, stream=None):
    _check(lib.coded_layer_step(plan.handle, phases, _ptr(W_shares), _ptr(X, _F32), _ptr(Delta, _F32), _ptr(DeltaT, _F32),
                                activation, eta, lam, inject_seed & 0xFFFFFFFFFFFFFFFF, inject_prob, inject_scale,
                                _ptr(S_out), _ptr(Xnext_out), _ptr(CT_out), _ptr(results), _ptr(workspace),
                                _stream(stream)), "coded_layer_step")


# ---- small helpers for callers --------------------------------------------------------------------
def new_results(count: int = 1, device="cuda") -> torch.Tensor:
    """Device buffer for `count` gpd_locate_result structs."""
    return torch.zeros(count * RESULT_BYTES, dtype=torch.uint8, device=device)


def read_results(buf: torch.Tensor):
    """Copies result structs back to the host (synchronises)."""
    raw = buf.cpu().numpy().tobytes()
    return [gpd_locate_result.from_buffer_copy(raw[i * RESULT_BYTES:(i + 1) * RESULT_BYTES])
            for i in range(len(raw) // RESULT_BYTES)]


def result_slot(buf: torch.Tensor, index: int) -> torch.Tensor:
    return buf[index * RESULT_BYTES:(index + 1) * RESULT_BYTES]
