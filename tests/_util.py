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


def block_rel_l2(got, want, ncols, block_rows=128, block_cols=256):
    """Largest relative L2 error over the block_rows x block_cols blocks of the (len / ncols) x ncols view
    of two vectors: a wrong strip at a ragged tile edge, or one misplaced output tile, cannot hide in the
    norm of the whole gradient.  Blocks follow the kernels' output tiling (128 rows x 256 columns)."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, ncols)
    want = np.asarray(want, dtype=np.float64).reshape(-1, ncols)
    worst = 0.0
    for r0 in range(0, got.shape[0], block_rows):
        for c0 in range(0, ncols, block_cols):
            g, w = got[r0:r0 + block_rows, c0:c0 + block_cols], want[r0:r0 + block_rows, c0:c0 + block_cols]
            worst = max(worst, float(np.linalg.norm(g - w) / max(np.linalg.norm(w), 1e-300)))
    return worst


def max_abs_scaled(got, want):
    """Largest absolute error relative to the largest magnitude of the expected values."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    return float(np.max(np.abs(got - want)) / max(np.max(np.abs(want)), 1e-300))


def assert_dense_close(got, want, ncols, tol, what="", max_abs=True):
    """Whole-vector relative L2, every 128 x 256 block of the matrix view, and (max_abs) the largest single error."""
    assert np.isfinite(np.asarray(got)).all(), what
    e = rel_l2(got, want)
    assert e < tol, (what, "rel L2", e)
    b = block_rel_l2(got, want, ncols)
    assert b < tol, (what, "worst 128 x 256 block", b)
    if max_abs:
        m = max_abs_scaled(got, want)
        assert m < tol, (what, "max abs / max |want|", m)
