"""Writes tests/golden/select_unit_small.json: the oracle's results on one small seeded case, two consecutive
events with the EMA credit carried.  Calls only `oracle/` (and numpy for the seeded scores); the stored values
guard the oracle against accidental changes and give the GPU tests an expected result that no GPU produced.
The paper prints no worked numeric example, so nothing here is a value from the paper.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402

T, TK, APPEND = 300, 64, 40
PRM = dict(n_segments=6, l_min=8, l_max=64, q_min=1, n_sink=2, n_last=5, ema_lambda=0.9, ema_beta=0.75, eps=1e-8)


def scores(event, n):
    rng = np.random.default_rng(20260523 + event)
    x = np.exp(1.5 * rng.standard_normal(n)).astype(np.float32)
    x[rng.integers(0, n, size=5)] = np.float32(0.25)         # a few exact ties
    return x


def main():
    prm = oracle.Params(**PRM)
    out = {"T": T, "Tk": TK, "append": APPEND, "params": PRM, "events": []}
    credit = np.zeros(T, np.float32)
    n = T
    for event in range(2):
        u = scores(event, n)
        r = oracle.select_unit(u, u, credit[:n], TK, prm)
        out["events"].append({
            "n_tokens": n, "n_seg": int(r.n_seg), "raw_bounds": r.raw_bounds.tolist(), "bounds": r.bounds.tolist(),
            "quotas": r.quotas.tolist(), "keep_idx": r.keep_idx.tolist(), "n_backfill": int(r.n_backfill),
            "mass_bits_first8": [int(v) for v in r.mass[:8].view(np.uint32)],
            "credit_bits_first8": [int(v) for v in r.credit[:8].view(np.uint32)],
            "credit_sum_f64": float(r.credit.astype(np.float64).sum())})
        credit = np.zeros(TK + APPEND, np.float32)
        credit[:TK] = r.credit[:TK]                            # rows travel with their tokens; new tokens start at zero
        n = TK + APPEND
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "select_unit_small.json"), "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")


if __name__ == "__main__":
    main()
