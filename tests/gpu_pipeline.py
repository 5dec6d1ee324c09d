"""Helpers for the GPU parity tests: run the coded product through the C ABI, stage by stage."""

from __future__ import annotations

import numpy as np
import torch

import paper_1811_10751_b200 as g
from oracle.code import GPCode


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def make_code(cfg, d2: int = 1) -> GPCode:
    return GPCode(cfg.N1, cfg.N0, cfg.B, cfg.m, cfg.n, cfg.d, d2, cfg.P)


class CodedProduct:
    """One plan plus the device buffers of a forward (and optionally backward) product."""

    def __init__(self, code: GPCode, precision: int = g.GPD_PREC_AUTO):
        self.code = code
        self.plan = g.gpd_plan((code.N1, code.N0, code.B), (code.m, code.n, code.d1, code.d2), code.P,
                               points=code.points, precision=precision, subst=code.subst)
        self.np_dtype = np.float32 if self.plan.query(g.GPD_Q_ELEMENT_SIZE) == 4 else np.float64
        self.ws = self.plan.workspace()
        self.res = g.new_results(1)
        self.W_shares = None

    # ---- stages --------------------------------------------------------------------------------
    def encode_W(self, W: np.ndarray) -> torch.Tensor:
        self.W_shares = self.plan.empty(g.GPD_Q_W_SHARE_ELEMS)
        g.gpd_encode_A(self.plan, dev(W), self.W_shares)
        return self.W_shares

    def encode(self, operand: int, M: np.ndarray) -> torch.Tensor:
        what = {g.GPD_OPERAND_X_FWD: g.GPD_Q_X_SHARE_ELEMS, g.GPD_OPERAND_DELTAT_BWD: g.GPD_Q_DT_SHARE_ELEMS,
                g.GPD_OPERAND_DELTA_UPD: g.GPD_Q_DHAT_ELEMS, g.GPD_OPERAND_X_UPD: g.GPD_Q_XHAT_ELEMS}[operand]
        sh = self.plan.empty(what)
        g.gpd_encode_B(self.plan, operand, dev(M), sh)
        return sh

    def products(self, which: int, other: torch.Tensor) -> torch.Tensor:
        out = self.plan.empty(g.GPD_Q_OUT_ELEMS_FWD if which == g.GPD_FWD else g.GPD_Q_OUT_ELEMS_BWD)
        out.fill_(float("nan"))                          # unwritten entries would show up in parity
        g.gpd_worker_gemm(self.plan, which, self.W_shares, other, out)
        return out

    def locate(self, which: int, Z: torch.Tensor, erased=None):
        g.gpd_locate_errors(self.plan, which, Z, self.res, self.ws, erased=erased)
        return g.read_results(self.res)[0]

    def decode(self, which: int, Z: torch.Tensor, use_mask=None, activation: int = g.GPD_ACT_IDENTITY,
               want_act: bool = False, fill: float = float("nan")):
        rows, cols = {g.GPD_FWD: (self.code.N1, self.code.B), g.GPD_BWD: (self.code.B, self.code.N0),
                      g.GPD_AUDIT: (self.code.N1, self.code.N0)}[which]
        out = torch.full((rows, cols), fill, dtype=torch.float32, device="cuda")
        act = torch.full((rows, cols), fill, dtype=torch.float32, device="cuda") if want_act else None
        g.gpd_decode(self.plan, which, Z, out, self.ws, result=None if use_mask is not None else self.res,
                     use_mask=use_mask, act_out=act, activation=activation)
        return (host(out), host(act)) if want_act else host(out)

    def outputs_as_array(self, which: int, Z: torch.Tensor) -> np.ndarray:
        br, bc = self.code.out_block_shape(which)
        return host(Z).reshape(self.code.P, br, bc)

    def flags(self, r) -> np.ndarray:
        return np.array(list(r.flagged)[: self.code.P], dtype=bool)
