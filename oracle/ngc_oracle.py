"""CPU oracle for the nested gradient code (NGC) hot path -- TEST INFRASTRUCTURE ONLY.

This module is a plain, slow, fp64 restatement of what the nested gradient
code of arXiv 2212.08580 computes.  It exists so that the CUDA library can be
checked against something written independently of it.  It shares no code
with the CUDA path and must never be imported by the product package; only
tests, the smoke check and the CPU-baseline leg of the benchmark call it.

Every function names the passage of the paper it follows.  Indices are
0-based and taken mod n; the paper's are 1-based.

Pin status (what each part is checked against in the CPU test-suite):
  * SplitMix64 stream ............ published test vector of the generator
  * supports / schedule .......... Definition 1 (row weight), Definition 2
                                   (nesting), Lemma 1 (cyclic windows)
  * coefficient VALUES of B ...... parity unpinned against the paper (it
                                   prints no example matrix); pinned only by
                                   the invariants of Definition 1 (rank,
                                   all-ones vector in every span, a.B = 1 on
                                   every straggler subset by brute force)
  * decode vector ................ uniqueness + residual + exact rational solve
  * selection rule ............... Lemma 2 / Theorem 1 closed forms (Monte
                                   Carlo), the 0.95^8 ceiling of Section III,
                                   Observation 1 load bound, hand cases
  * partial gradients ............ finite differences of the loss, autograd,
                                   normal equations; the optional ReLU decision
                                   of grad_mlp: identity with the default when
                                   handed the default's own decision, a 2 x 2
                                   case worked by hand, the all-ones mask
  * decoded gradient ............. equals the plain full-data gradient
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# Counter-based generator: SplitMix64 (Steele, Lea, Flood, "Fast splittable
# pseudorandom number generators", OOPSLA 2014; Vigna's public-domain
# splitmix64.c).  Output number k (k = 1, 2, ...) of the stream seeded with
# `seed` is mix(seed + k * GOLDEN).
# --------------------------------------------------------------------------
_MASK = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15


def splitmix64_at(seed: int, k: int) -> int:
    z = (seed + k * _GOLDEN) & _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def h_entry(seed: int, sigma: int, r: int, c: int) -> float:
    """Entry (r, c), c < n-1, of the auxiliary matrix H of the sigma-code.

    The paper is silent on how the coefficients are drawn (Algorithm 1 defers
    to determineCoef of the gradient-coding paper it cites).  Reading used
    here: a dyadic uniform in [-1, 1) taken from the top 53 bits of stream
    position 1 + (sigma * 2^20 + r * 2^10 + c), so that two programs can
    agree bit for bit without transcendental functions.
    """
    k = 1 + ((sigma << 20) | (r << 10) | c)
    u = splitmix64_at(seed, k) >> 11          # 53 bits
    return u / 4503599627370496.0 - 1.0       # u / 2^52 - 1, exact in fp64


# --------------------------------------------------------------------------
# Supports and schedule (Definition 2; Lemma 1; "layered task scheduling" of
# Section III).
# --------------------------------------------------------------------------
def window(n: int, sigma: int, i: int) -> list[int]:
    """supp(b_sigma^(i)) = {i, i+1, ..., i+sigma} mod n (sigma+1 entries).

    Lemma 1 prints a window one entry longer; that contradicts B_0 = I in the
    same proof and the row weight (k/n)(sigma+1) of Definition 1, so the
    minimum-load reading is taken.
    """
    return [(i + t) % n for t in range(sigma + 1)]


def schedule(n: int, levels: list[int]) -> np.ndarray:
    """Task order of every worker: its widest window read left to right.

    Worker i has finished component code s_l once its first s_l+1 tasks are
    done (Section III, task scheduling).
    """
    s_max = levels[-1]
    return np.array([window(n, s_max, i) for i in range(n)], dtype=np.int32)


# --------------------------------------------------------------------------
# Coefficients (Algorithm 1: B_0 = I; B_sigma = determineCoef(n, sigma)).
# --------------------------------------------------------------------------
def _aux_matrix(n: int, sigma: int, seed: int) -> np.ndarray:
    """H in R^{sigma x n} with every row summing to zero (so H 1 = 0)."""
    H = np.zeros((sigma, n))
    for r in range(sigma):
        acc = 0.0
        for c in range(n - 1):
            H[r, c] = h_entry(seed, sigma, r, c)
            acc = acc + H[r, c]               # left-to-right
        H[r, n - 1] = -acc
    return H


def _solve_gepp(M: np.ndarray, rhs: np.ndarray) -> np.ndarray:
    """Gaussian elimination with partial pivoting in a fixed operation order.

    Pivot = first row of maximal |entry| in the column; elimination row by
    row, columns increasing; back substitution from the last unknown, columns
    increasing.  Python floats: one rounding per operation, no fused
    multiply-add.
    """
    s = len(rhs)
    M = [[float(M[r, c]) for c in range(s)] for r in range(s)]
    b = [float(v) for v in rhs]
    for p in range(s):
        best, q = abs(M[p][p]), p
        for r in range(p + 1, s):
            if abs(M[r][p]) > best:
                best, q = abs(M[r][p]), r
        if q != p:
            M[p], M[q] = M[q], M[p]
            b[p], b[q] = b[q], b[p]
        for r in range(p + 1, s):
            f = M[r][p] / M[p][p]
            for c in range(p + 1, s):
                M[r][c] = M[r][c] - f * M[p][c]
            b[r] = b[r] - f * b[p]
    z = [0.0] * s
    for p in range(s - 1, -1, -1):
        acc = b[p]
        for c in range(p + 1, s):
            acc = acc - M[p][c] * z[c]
        z[p] = acc / M[p][p]
    return np.array(z)


def coefficients(n: int, sigma: int, seed: int) -> np.ndarray:
    """Dense B_sigma in R^{n x n} (k = n).

    sigma = 0 gives the identity (Algorithm 1, initialisation).  Otherwise
    row i has b_ii = 1 and its other sigma window entries chosen so that
    H b_i^T = 0: all rows then lie in null(H), an (n-sigma)-dimensional space
    that contains the all-ones vector, which is what Definition 1 asks of
    every n-sigma rows.
    """
    B = np.zeros((n, n))
    if sigma == 0:
        for i in range(n):
            B[i, i] = 1.0
        return B
    H = _aux_matrix(n, sigma, seed)
    for i in range(n):
        cols = window(n, sigma, i)
        z = _solve_gepp(H[:, cols[1:]], -H[:, cols[0]])
        B[i, cols[0]] = 1.0
        for t in range(sigma):
            B[i, cols[t + 1]] = z[t]
    return B


def plan(n: int, levels: list[int], seed: int) -> dict:
    """Component codes of the NGC restricted to the listed tolerances.

    The paper nests every sigma = 0..s_max (Definition 2); a strictly
    increasing subset s_1 < ... < s_L is the same construction with the
    unlisted components left out.
    """
    assert all(0 <= s < n for s in levels)
    assert all(a < b for a, b in zip(levels, levels[1:]))
    return {
        "n": n,
        "levels": list(levels),
        "B": [coefficients(n, s, seed) for s in levels],
        "schedule": schedule(n, levels),
        "tasks_per_level": np.array([s + 1 for s in levels], dtype=np.int32),
    }


# --------------------------------------------------------------------------
# Stopping and signalling rule (Section II-D last paragraph, Section III last
# paragraph, proof of Theorem 1).
# --------------------------------------------------------------------------
def select(times: np.ndarray, levels: list[int], gamma: float, eps: float):
    """Which component code the main node terminates on, and with whom.

    times[i, m] is the duration of worker i's (m+1)-th task (+inf = never).
    C_i(u) = completion instant of u tasks, added left to right.  Component
    s_l is decodable at the instant D_l when n - s_l workers have finished
    s_l + 1 tasks.  The main node stops at the first such instant; ties go to
    the smaller level index.  Exactly n - s_l responders are used (the
    earliest, ties by worker index), so the decoding vector is unique.
    Returns None when no component ever becomes decodable.
    """
    n, n_tasks = times.shape
    assert n_tasks == levels[-1] + 1
    C = np.zeros((n, n_tasks))
    for i in range(n):
        acc = 0.0
        for m in range(n_tasks):
            acc = acc + float(times[i, m])
            C[i, m] = acc
    best_l, best_D = -1, np.inf
    for l, s in enumerate(levels):
        col = sorted(C[i, s] for i in range(n))
        D = col[n - s - 1]
        if D < best_D:
            best_l, best_D = l, D
    if best_l < 0:
        return None
    s = levels[best_l]
    order = sorted(range(n), key=lambda i: (C[i, s], i))
    S = sorted(order[: n - s])
    done = np.zeros(n, dtype=np.int32)
    for i in range(n):
        for m in range(n_tasks):
            if C[i, m] <= best_D:
                done[i] = m + 1
    return {
        "level": best_l,
        "sigma": s,
        "S": np.array(S, dtype=np.int32),
        "latency": gamma + eps + best_D,
        "tasks_done": done,
    }


# --------------------------------------------------------------------------
# Partial gradients (Section II-C: g_j = sum over the rows of partition j of
# the per-sample loss gradient; a sum, not a mean -- the 1/m sits in Eq. 1).
# The paper fixes no loss; the four below are the textbook ones.
# --------------------------------------------------------------------------
def grad_lsq(X, y, theta):
    """L = 1/2 (x.theta - y)^2  ->  X^T (X theta - y)."""
    X = np.asarray(X, dtype=np.float64)
    r = X @ np.asarray(theta, dtype=np.float64) - np.asarray(y, dtype=np.float64)
    return X.T @ r


def grad_logistic(X, y, theta):
    """Binary cross-entropy with labels in {0,1}  ->  X^T (sigmoid(X theta) - y)."""
    X = np.asarray(X, dtype=np.float64)
    z = X @ np.asarray(theta, dtype=np.float64)
    p = 1.0 / (1.0 + np.exp(-z))
    return X.T @ (p - np.asarray(y, dtype=np.float64))


def _softmax_rows(Z):
    Z = Z - Z.max(axis=1, keepdims=True)
    E = np.exp(Z)
    return E / E.sum(axis=1, keepdims=True)


def grad_softmax(X, labels, W):
    """Multinomial cross-entropy, W in R^{d x C}  ->  X^T (softmax(X W) - onehot), flattened row-major."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    P = _softmax_rows(X @ W)
    P[np.arange(X.shape[0]), np.asarray(labels)] -= 1.0
    return (X.T @ P).reshape(-1)


def mlp_unpack(theta, d, hidden, n_classes):
    theta = np.asarray(theta, dtype=np.float64)
    o = 0
    W1 = theta[o:o + d * hidden].reshape(d, hidden); o += d * hidden
    b1 = theta[o:o + hidden]; o += hidden
    W2 = theta[o:o + hidden * n_classes].reshape(hidden, n_classes); o += hidden * n_classes
    b2 = theta[o:o + n_classes]; o += n_classes
    assert o == theta.size
    return W1, b1, W2, b2


def grad_mlp(X, labels, theta, hidden, n_classes, relu_mask=None):
    """One-hidden-layer ReLU network with softmax cross-entropy, back-propagated.

    Parameters flattened as [W1 (d x hidden, row-major), b1, W2 (hidden x C), b2];
    ReLU'(0) = 0.  `relu_mask` (rows x hidden, 0/1), when given, replaces the
    derivative decision pre > 0: that decision is an integer taken from floating
    point, and a checker may want both sides to take it in the same precision.
    Everything else stays fp64.
    """
    X = np.asarray(X, dtype=np.float64)
    d = X.shape[1]
    W1, b1, W2, b2 = mlp_unpack(theta, d, hidden, n_classes)
    pre = X @ W1 + b1
    h = np.maximum(pre, 0.0)
    P = _softmax_rows(h @ W2 + b2)
    P[np.arange(X.shape[0]), np.asarray(labels)] -= 1.0      # delta2
    dW2 = h.T @ P
    db2 = P.sum(axis=0)
    delta1 = (P @ W2.T) * ((pre > 0.0) if relu_mask is None else np.asarray(relu_mask, dtype=np.float64))
    dW1 = X.T @ delta1
    db1 = delta1.sum(axis=0)
    return np.concatenate([dW1.reshape(-1), db1, dW2.reshape(-1), db2])


def partial_gradient(kind: str, X, y, theta, hidden: int = 0, n_classes: int = 0):
    if kind == "lsq":
        return grad_lsq(X, y, theta)
    if kind == "logistic":
        return grad_logistic(X, y, theta)
    if kind == "softmax":
        d = np.asarray(X).shape[1]
        return grad_softmax(X, y, np.asarray(theta).reshape(d, n_classes))
    if kind == "mlp":
        return grad_mlp(X, y, theta, hidden, n_classes)
    raise ValueError(kind)


def partial_gradients(kind, X_parts, y_parts, theta, hidden=0, n_classes=0):
    """G = (g_1, ..., g_k)^T in R^{k x l} (Section II-C)."""
    return np.stack([partial_gradient(kind, X_parts[j], y_parts[j], theta, hidden, n_classes)
                     for j in range(len(X_parts))])


def full_gradient(kind, X_parts, y_parts, theta, hidden=0, n_classes=0):
    """The plain definition g = sum over ALL samples (Eq. 1), no partitioning, no code."""
    X = np.concatenate([np.asarray(x, dtype=np.float64) for x in X_parts], axis=0)
    y = np.concatenate([np.asarray(v) for v in y_parts], axis=0)
    return partial_gradient(kind, X, y, theta, hidden, n_classes)


# --------------------------------------------------------------------------
# Encode / decode (Section II-C: X = B G; Definition 1: a B = 1 with
# supp(a) inside the responsive set).
# --------------------------------------------------------------------------
def encode(B: np.ndarray, G: np.ndarray) -> np.ndarray:
    """Worker responses x_i = b^(i) G, all workers at once."""
    return B @ G


def decode_vector(B: np.ndarray, S) -> np.ndarray:
    """Row a of the decoding matrix for responsive set S: supp(a) in S, a B = 1.

    The n equations (one per partition) in |S| unknowns are consistent; the
    least-squares routine returns the exact solution, unique when |S| = n - sigma.
    """
    S = list(S)
    n = B.shape[0]
    sol, *_ = np.linalg.lstsq(B[S, :].T, np.ones(n), rcond=None)
    a = np.zeros(n)
    a[S] = sol
    return a


def decode(a: np.ndarray, coded: np.ndarray) -> np.ndarray:
    """Main node's g = sum_{i in S} a_i x_i (a is zero off S)."""
    idx = np.nonzero(a)[0]
    g = np.zeros(coded.shape[1])
    for i in idx:
        g = g + a[i] * coded[i]
    return g


def step(pl: dict, kind, X_parts, y_parts, theta, times, gamma, eps, hidden=0, n_classes=0):
    """One iteration: select -> partial gradients -> encode at the chosen component -> decode."""
    sel = select(np.asarray(times, dtype=np.float64), pl["levels"], gamma, eps)
    if sel is None:
        return None
    B = pl["B"][sel["level"]]
    G = partial_gradients(kind, X_parts, y_parts, theta, hidden, n_classes)
    coded = encode(B, G)
    a = decode_vector(B, sel["S"])
    sel["a"] = a
    sel["coded"] = coded
    sel["grad"] = decode(a, coded)
    return sel
