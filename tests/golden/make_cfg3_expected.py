"""Writes tests/golden/cfg3_full_expected.json: what the oracle decides on the full-size
8192 x 8192 x 512 coded product (the benchmark workload) for each injection seed.

Calls only oracle/ and workloads/.  Takes about a minute and 5 GB of host memory:
    python tests/golden/make_cfg3_expected.py
"""

import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import workloads as wl                                    # noqa: E402
from oracle import inject as oinj                         # noqa: E402
from oracle import product as op                          # noqa: E402
from oracle.code import GPCode, FWD                       # noqa: E402
from oracle.locate import locate_subspace, tolerances_for  # noqa: E402


def main():
    cfg = wl.CONFIG_3_MATMUL
    W, X = wl.matmul_inputs(cfg)
    code = GPCode(cfg.N1, cfg.N0, cfg.B, cfg.m, cfg.n, cfg.d, 1, cfg.P)
    Z = op.worker_products(op.encode_W(W, code), op.encode_X(X, code))
    scale = float(np.sqrt(np.mean(Z * Z)))
    rng = np.random.default_rng(12345)
    L = Z[0].size
    sample_pos = sorted(int(v) for v in rng.choice(L, size=48, replace=False))
    out = {"config": cfg.name, "scale": scale, "sample_positions": sample_pos,
           "clean_outputs_at_samples": Z.reshape(cfg.P, L)[:, sample_pos].tolist(), "seeds": {}}
    ref = op.ref_forward(W, X)
    for seed in cfg.inject_seeds:
        Zr = Z.copy()
        sel = oinj.inject_additive(Zr, seed, scale, prob=cfg.inject_prob)
        r = locate_subspace(Zr, code.points, code.Q_f, tolerances_for(np.float64))
        entry = {"injected": np.flatnonzero(sel).tolist(), "outcome": int(r.outcome),
                 "flagged": np.flatnonzero(r.flagged).tolist(), "rank": int(r.rank), "n_active": int(r.n_active)}
        if r.outcome != 2:
            S = op.decode(Zr, code, FWD, use=~r.flagged)
            entry["rel_err_vs_uncoded"] = op.rel_fro(S, ref)
        out["seeds"][str(seed)] = entry
        print(seed, entry)
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg3_full_expected.json"), "w") as f:
        json.dump(out, f, indent=1)


if __name__ == "__main__":
    main()
