"""Seeded synthetic inputs for the nested-gradient-code hot path.

This module only draws random numbers and shapes them; it contains none of
the method's arithmetic (no gradients, no code construction, no selection),
so both the CUDA library's callers and the CPU oracle's callers may use it.

Five workloads mirror the shapes the method is measured on; `scale` shrinks
the per-partition row count (and, for "d_scale", the feature count) so that
the CPU oracle finishes in seconds.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np
import torch

BASE_SEED = 221208580


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # seed offset
    n: int                     # workers = partitions
    levels: tuple              # straggler tolerances s_1 < ... < s_L
    kind: str                  # "lsq" | "logistic" | "softmax" | "mlp"
    rows: int                  # rows per partition
    d: int                     # features
    x_dtype: str               # "f32" | "bf16"
    n_classes: int = 0
    hidden: int = 0
    pattern: str = "times"     # "times" (shifted exponential) | "sets" (fixed straggler sets)
    p_fail: float = 0.0
    unit_x: bool = False       # X ~ N(0,1) instead of N(0,1/d)

    @property
    def n_params(self) -> int:
        if self.kind in ("lsq", "logistic"):
            return self.d
        if self.kind == "softmax":
            return self.d * self.n_classes
        return self.d * self.hidden + self.hidden + self.hidden * self.n_classes + self.n_classes

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


WORKLOADS = {
    "tiny": Workload("tiny", 0, 4, (1, 2), "lsq", 64, 32, "f32", pattern="sets", unit_x=True),
    "logistic20": Workload("logistic20", 1, 20, (1, 2, 4), "logistic", 8192, 4096, "f32"),
    "softmax50": Workload("softmax50", 2, 50, (1, 3, 5, 10), "softmax", 4096, 1024, "bf16",
                          n_classes=256, pattern="sets"),
    "lsq100": Workload("lsq100", 3, 100, (1, 2, 5, 10), "lsq", 2000, 16384, "bf16", p_fail=0.05),
    "mlp30": Workload("mlp30", 4, 30, (1, 2, 3, 6), "mlp", 2000, 784, "f32",
                      n_classes=10, hidden=512, pattern="sets"),
}


def shrink(w: Workload, rows: int | None = None, d: int | None = None) -> Workload:
    return replace(w, rows=rows if rows is not None else w.rows, d=d if d is not None else w.d)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_data(w: Workload, device="cpu"):
    """Returns (X, y, theta) as torch tensors on `device`.

    X: [n, rows, d] in the workload's storage dtype; y: [n, rows] fp32
    (regression targets or 0/1 labels) or int32 class ids; theta: [l] fp32.
    Partitions are generated one at a time so that the full-size workloads
    never hold an fp32 copy of a bf16 data matrix.
    """
    dev = torch.device(device)
    g = _gen(w.seed, dev)
    xdt = torch.bfloat16 if w.x_dtype == "bf16" else torch.float32
    X = torch.empty((w.n, w.rows, w.d), dtype=xdt, device=dev)
    if w.kind in ("lsq", "logistic"):
        std = 1.0 if w.unit_x else 1.0 / math.sqrt(w.d)
        theta_star = torch.randn(w.d, generator=g, device=dev)
        theta = torch.randn(w.d, generator=g, device=dev)
        y = torch.empty((w.n, w.rows), dtype=torch.float32, device=dev)
        for j in range(w.n):
            xj = (torch.randn((w.rows, w.d), generator=g, device=dev) * std).to(xdt)
            X[j] = xj
            z = xj.float() @ theta_star
            if w.kind == "lsq":
                y[j] = z + 0.1 * torch.randn(w.rows, generator=g, device=dev)      # N(0, 0.01): variance
            else:
                y[j] = (torch.rand(w.rows, generator=g, device=dev) < torch.sigmoid(z)).float()
        return X, y, theta
    if w.kind == "softmax":
        for j in range(w.n):
            X[j] = (torch.randn((w.rows, w.d), generator=g, device=dev) / math.sqrt(w.d)).to(xdt)
        y = torch.randint(0, w.n_classes, (w.n, w.rows), generator=g, device=dev, dtype=torch.int32)
        theta = 0.1 * torch.randn(w.d * w.n_classes, generator=g, device=dev)       # N(0, 0.01)
        return X, y, theta
    if w.kind == "mlp":
        for j in range(w.n):
            X[j] = torch.rand((w.rows, w.d), generator=g, device=dev).to(xdt)
        y = torch.randint(0, w.n_classes, (w.n, w.rows), generator=g, device=dev, dtype=torch.int32)
        W1 = torch.randn(w.d * w.hidden, generator=g, device=dev) * math.sqrt(2.0 / w.d)
        W2 = torch.randn(w.hidden * w.n_classes, generator=g, device=dev) * math.sqrt(2.0 / w.hidden)
        theta = torch.cat([W1, torch.zeros(w.hidden, device=dev), W2, torch.zeros(w.n_classes, device=dev)])
        return X, y, theta
    raise ValueError(w.kind)


def make_data_batched(w: Workload, device="cpu"):
    """Same distributions as `make_data`, all partitions drawn by one call per tensor (a handful of
    launches on a GPU).  For small cases only: the whole data matrix exists in fp32 for a moment.  The
    values differ from `make_data`'s for the same seed (the generator is consumed in another order)."""
    dev = torch.device(device)
    g = _gen(w.seed, dev)
    xdt = torch.bfloat16 if w.x_dtype == "bf16" else torch.float32
    shape = (w.n, w.rows, w.d)
    if w.kind in ("lsq", "logistic"):
        std = 1.0 if w.unit_x else 1.0 / math.sqrt(w.d)
        theta_star = torch.randn(w.d, generator=g, device=dev)
        theta = torch.randn(w.d, generator=g, device=dev)
        X = (torch.randn(shape, generator=g, device=dev) * std).to(xdt)
        z = X.float() @ theta_star
        if w.kind == "lsq":
            y = z + 0.1 * torch.randn((w.n, w.rows), generator=g, device=dev)
        else:
            y = (torch.rand((w.n, w.rows), generator=g, device=dev) < torch.sigmoid(z)).float()
        return X, y, theta
    y = torch.randint(0, w.n_classes, (w.n, w.rows), generator=g, device=dev, dtype=torch.int32)
    if w.kind == "softmax":
        X = (torch.randn(shape, generator=g, device=dev) / math.sqrt(w.d)).to(xdt)
        return X, y, 0.1 * torch.randn(w.d * w.n_classes, generator=g, device=dev)
    if w.kind == "mlp":
        X = torch.rand(shape, generator=g, device=dev).to(xdt)
        theta = torch.zeros(w.n_params, device=dev)
        o = w.d * w.hidden
        theta[:o] = torch.randn(o, generator=g, device=dev) * math.sqrt(2.0 / w.d)
        o2 = o + w.hidden
        theta[o2:o2 + w.hidden * w.n_classes] = (torch.randn(w.hidden * w.n_classes, generator=g, device=dev)
                                                 * math.sqrt(2.0 / w.hidden))
        return X, y, theta
    raise ValueError(w.kind)


def sample_times(n: int, n_tasks: int, seed: int, shift=1.0, rate=1.0, p_fail=0.0) -> np.ndarray:
    """Per-task durations [n, n_tasks]: shift + Exp(rate) i.i.d.; a worker fails
    (all its tasks +inf) independently with probability p_fail."""
    rng = np.random.default_rng(seed)
    t = shift + rng.exponential(1.0 / rate, size=(n, n_tasks))
    dead = rng.random(n) < p_fail
    t[dead, :] = np.inf
    return t


def set_times(n: int, n_tasks: int, stragglers) -> np.ndarray:
    """A fixed straggler set written as task times: stragglers never finish,
    everyone else takes one time unit per task."""
    t = np.ones((n, n_tasks))
    for i in stragglers:
        t[int(i), :] = np.inf
    return t


def sample_set(n: int, size: int, seed: int) -> list[int]:
    rng = np.random.default_rng(seed)
    return sorted(int(v) for v in rng.choice(n, size=size, replace=False))


def pattern_times(w: Workload, it: int) -> np.ndarray:
    """The it-th straggler pattern of a workload, as a task-time matrix."""
    n_tasks = w.levels[-1] + 1
    seed = w.seed * 1000003 + it
    if w.pattern == "times":
        return sample_times(w.n, n_tasks, seed, 1.0, 1.0, w.p_fail)
    size = it % (w.levels[-1] + 1)          # sweep actual straggler counts 0..s_L
    return set_times(w.n, n_tasks, sample_set(w.n, size, seed))
