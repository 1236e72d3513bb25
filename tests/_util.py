"""Shared helpers for the parity tests: run the CPU oracle on the very bits the GPU gets."""
import numpy as np
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc


def to_np64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of fp32 / bf16 / int tensors to numpy (fp64 for floats)."""
    t = t.detach().cpu()
    if t.dtype in (torch.float32, torch.bfloat16):
        return t.to(torch.float64).numpy()
    return t.numpy()


def model_of(w: ngc_inputs.Workload) -> ngc.Model:
    return ngc.Model.make(w.kind, w.x_dtype, w.rows, w.d, w.n_classes, w.hidden)


def oracle_G(w, X, y, theta):
    """Partial gradients of every partition, one partition at a time (fp64)."""
    th = to_np64(theta)
    return np.stack([orc.partial_gradient(w.kind, to_np64(X[j]), to_np64(y[j]), th, w.hidden, w.n_classes)
                     for j in range(X.shape[0])])


def group_G(G, q):
    """k = q n: an atomic task is q consecutive partitions (Section II-C)."""
    if q == 1:
        return G
    return G.reshape(G.shape[0] // q, q, -1).sum(axis=1)


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def coded_torch_dtype(code: int):
    return torch.float64 if code == ngc.NGC_F64 else torch.float32
