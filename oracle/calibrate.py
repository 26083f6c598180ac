"""Writes ``dsmoe_inputs/calibration.json``: the two scalars that shape the synthetic
workloads so that 30-40 % of experts are active per token, the range the paper reports for
DS-MoE at inference (abstract; "Active Hidden" column of the zero-shot results table).

TEST INFRASTRUCTURE: calls only the CPU oracle and the input generator.

  c1_router_gain  scalar on the drawn Wr of the tiny fp32 layer such that the mean fraction
                  of experts with raw score > 0.1 is 0.35
  c2_eps          raw-score threshold of the decode-shaped layer such that the mean active
                  fraction over a 4096-token calibration batch is 0.35

Run:  python -m oracle.calibrate
"""
import json
import os

import numpy as np

import dsmoe_inputs as gi
import oracle


def active_fraction(s, batch, T):
    s = s.replace(T=T)
    x = gi.tokens(s, batch)
    Wr, br = gi.router(s)
    S = oracle.router_scores(x, Wr, br)
    _, k_t = oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
    return float(k_t.mean()) / s.E


def bisect(f, lo, hi, target, iters=60):
    """f decreasing in its argument; returns the argument with f closest to target."""
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if f(mid) > target:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def main():
    base1 = gi.LayerSpec("c1", T=64, d=256, H=512, E=8, dtype="f32", mode=gi.MODE_THRESHOLD, eps=0.1)
    g = bisect(lambda gain: active_fraction(base1.replace(router_gain=gain), "x", 64), 0.1, 50.0, 0.35)
    g = float(np.float32(round(g, 3)))
    base2 = gi.LayerSpec("c2", T=4096, d=2048, H=1024, E=32, dtype="bf16", mode=gi.MODE_THRESHOLD)
    eps = bisect(lambda e: active_fraction(base2.replace(eps=e), "calib", 4096), 0.0, 1.0, 0.35)
    eps = float(np.float32(round(eps, 5)))
    out = {"c1_router_gain": g, "c2_eps": eps,
           "c1_active_fraction": active_fraction(base1.replace(router_gain=g), "x", 64),
           "c2_active_fraction_calib": active_fraction(base2.replace(eps=eps), "calib", 4096)}
    path = os.path.join(os.path.dirname(os.path.abspath(gi.__file__)), "calibration.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")
    print(out)


if __name__ == "__main__":
    main()
