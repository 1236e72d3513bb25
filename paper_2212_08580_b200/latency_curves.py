"""Latency CDFs of Section IV for the settings of the paper's two figures (n = k = 8, lambda = 0.5, rho = 0.5,
eps = 0.1, p_e = 0.05, plotted against t - gamma).

    python -m paper_2212_08580_b200.latency_curves            # closed forms (Lemma 2, Theorem 1), host only
    python -m paper_2212_08580_b200.latency_curves --mc 1000000   # adds the GPU Monte Carlo of the stopping rule

Prints one table per figure: columns = schemes, rows = t - gamma.
"""
from __future__ import annotations

import argparse

import numpy as np

from . import Plan, latency_cdf_gc, latency_cdf_ngc

PARAMS = dict(n=8, lam=0.5, rho=0.5, eps=0.1, p_fail=0.05)
FIGURES = {
    "Fig. 1": [("GC", 0), ("GC", 3), ("NGC", 3)],
    "Fig. 2": [("GC", 1), ("GC", 2), ("GC", 4), ("GC", 6), ("NGC", 2), ("NGC", 4), ("NGC", 6)],
}


def closed_form(kind: str, s: int, t: float) -> float:
    f = latency_cdf_gc if kind == "GC" else latency_cdf_ngc
    return f(PARAMS["n"], s, t, PARAMS["lam"], PARAMS["rho"], 0.0, PARAMS["eps"], PARAMS["p_fail"])


def monte_carlo(kind: str, s: int, grid, trials: int):
    import torch
    levels = [s] if kind == "GC" else list(range(s + 1))
    plan = Plan(PARAMS["n"], levels, seed=1, gamma=0.0, eps=PARAMS["eps"])
    lat = torch.empty(trials, dtype=torch.float64, device="cuda")
    lev = torch.empty(trials, dtype=torch.int32, device="cuda")
    plan.latency_mc(12345 + 17 * s, PARAMS["rho"], PARAMS["lam"], PARAMS["p_fail"], lat, lev)
    torch.cuda.synchronize()
    lat = torch.sort(lat).values.cpu().numpy()
    return [float(np.searchsorted(lat, t, side="right")) / trials for t in grid]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mc", type=int, default=0, help="Monte-Carlo trials per scheme on the GPU (0 = closed forms only)")
    args = ap.parse_args()
    grid = np.arange(2.0, 18.5, 1.0)
    for fig, schemes in FIGURES.items():
        print(f"{fig}: P(T <= t), n = k = 8, lambda = 0.5, rho = 0.5, eps = 0.1, p_e = 0.05")
        head = "t-gamma " + " ".join(f"{k}{'s=' if k == 'GC' else 'smax='}{s:<2d}".rjust(12) for k, s in schemes)
        print(head)
        mc = {sc: monte_carlo(sc[0], sc[1], grid, args.mc) for sc in schemes} if args.mc else {}
        for gi, t in enumerate(grid):
            cells = []
            for sc in schemes:
                v = closed_form(sc[0], sc[1], t)
                cells.append(f"{v:.4f}" + (f"/{mc[sc][gi]:.4f}" if args.mc else ""))
            print(f"{t:7.1f} " + " ".join(c.rjust(12) for c in cells))
        print()


if __name__ == "__main__":
    main()
