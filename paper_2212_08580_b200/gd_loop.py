"""Gradient descent (Eq. 1) driven by a gradient code, with the latency of every iteration taken from the
straggler model of Section II-D: per-task times rho + Exp(lambda), a worker failing with probability p_e,
constants gamma and eps added once per iteration.

    python -m paper_2212_08580_b200.gd_loop --iters 50        # nested code vs fixed codes vs uncoded, least squares

Every scheme sees the same per-task times in the same iteration, so the latencies are directly comparable:
a nested code with levels 0..s_bar stops as early as the best fixed code of the iteration (Section III).
An iteration whose pattern no component code can decode (more hard stragglers than the largest tolerance) is
repeated with fresh times and its waiting time is not counted: the model's latency is infinite there.

Only argument marshalling happens here; gradients, encode, decode and update run in the CUDA library.
"""
from __future__ import annotations

import argparse
from dataclasses import dataclass, field

import numpy as np

from . import NgcError, Plan, gd_update, sample_times
from .binding import NGC_F64


@dataclass
class History:
    latency: list = field(default_factory=list)        # model time of every completed iteration
    level: list = field(default_factory=list)          # component code that decoded it
    tasks_done: list = field(default_factory=list)     # partial gradients computed by all workers together
    undecodable: int = 0                               # patterns that had to be redrawn

    @property
    def total_latency(self) -> float:
        return float(np.sum(self.latency))


def run(plan: Plan, model, theta, X, y, iters: int, step: float, seed: int, rho: float = 0.5, lam: float = 0.5,
        p_fail: float = 0.0, times_width: int | None = None, stream: int = 0) -> History:
    """`iters` iterations of theta <- theta - step * g on the device, g decoded by `plan` under a fresh seeded
    straggler pattern per iteration.  theta is updated in place; returns the latency record.

    `times_width` = tasks per worker that are drawn (default: what this plan needs).  Schemes that are to see the
    same times must be given the same width (the largest any of them needs); each reads the first columns."""
    import torch
    l = int(theta.numel())
    cdt = plan.coded_dtype(model)
    coded = torch.empty((plan.n, l), dtype=torch.float64 if cdt == NGC_F64 else torch.float32, device=theta.device)
    grad = torch.empty(l, dtype=torch.float32, device=theta.device)
    tasks = plan.levels[-1] + 1
    width = max(tasks, times_width or 0)
    hist = History()
    draw = 0
    for _ in range(iters):
        while True:
            t = sample_times(seed + draw, plan.n, width, rho, lam, p_fail)[:, :tasks]
            draw += 1
            try:
                info = plan.step(model, theta, X, y, np.ascontiguousarray(t), coded, grad, stream)
                break
            except NgcError as e:
                if e.status != -2:      # NGC_ERR_UNDECODABLE
                    raise
                hist.undecodable += 1
        gd_update(theta, grad, step, stream)
        hist.latency.append(info.latency)
        hist.level.append(info.layer)
        hist.tasks_done.append(int(sum(info.tasks_done[: plan.n])))
    return hist


def _main():
    import torch

    import ngc_inputs
    from . import Model

    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--iters", type=int, default=50)
    ap.add_argument("--n", type=int, default=8)
    ap.add_argument("--s-bar", type=int, default=3)
    ap.add_argument("--p-fail", type=float, default=0.0,
                    help="probability that a worker never responds; a redrawn iteration (column 'redrawn') had "
                         "infinite latency under that scheme and shifts its later draws")
    ap.add_argument("--seed", type=int, default=2212)
    args = ap.parse_args()
    w = ngc_inputs.Workload("gd_demo", 77, args.n, (0,), "lsq", 512, 256, "f32", unit_x=True)
    X, y, theta0 = ngc_inputs.make_data(w, "cuda")
    model = Model.make(w.kind, w.x_dtype, w.rows, w.d)
    step = 0.5 / (w.n * w.rows)
    schemes = [("nested 0..%d" % args.s_bar, list(range(args.s_bar + 1)))]
    schemes += [("fixed sigma=%d" % s, [s]) for s in range(args.s_bar + 1)]
    print(f"{'scheme':16s} {'total latency':>14s} {'mean':>8s} {'tasks/iter':>11s} {'redrawn':>8s} {'final loss':>12s}")
    for name, levels in schemes:
        plan = Plan(args.n, levels, seed=1, gamma=0.0, eps=0.1)
        theta = theta0.clone()
        h = run(plan, model, theta, X, y, args.iters, step, args.seed, p_fail=args.p_fail, times_width=args.s_bar + 1)
        torch.cuda.synchronize()
        r = (X.reshape(-1, w.d) @ theta - y.reshape(-1)).double()
        print(f"{name:16s} {h.total_latency:14.2f} {np.mean(h.latency):8.3f} {np.mean(h.tasks_done):11.1f} "
              f"{h.undecodable:8d} {0.5 * float(r @ r):12.4e}")


if __name__ == "__main__":
    _main()
