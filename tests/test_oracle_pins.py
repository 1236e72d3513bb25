"""Pins the CPU oracle to what the paper and the mathematics fix (no GPU).

Each test names the passage it checks.  None of them re-uses the oracle's own
formula as the expected value: the expectations are invariants of
Definition 1 / 2, closed forms of Section IV, library routines (exact
rationals, autograd, scipy distributions), brute force, or printed values.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import ngc_inputs
from oracle import latency, ngc_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SEED = 221208580


# ------------------------------------------------------------------ generator
def test_splitmix64_published_vector():
    # first five outputs for seed 1234567 (reference vector of the public-domain splitmix64.c)
    want = [6457827717110365317, 3203168211198807973, 9817491932198370423,
            4593380528125082431, 16408922859458223821]
    assert [orc.splitmix64_at(1234567, k) for k in range(1, 6)] == want


def test_h_entries_are_dyadic_in_range():
    vals = [orc.h_entry(SEED, s, r, c) for s in (1, 5, 10) for r in range(s) for c in range(99)]
    assert all(-1.0 <= v < 1.0 for v in vals)
    assert all(v * 2 ** 52 == int(v * 2 ** 52) for v in vals)
    assert abs(np.mean(vals)) < 0.05 and 0.28 < np.var(vals) < 0.39      # uniform[-1,1): var 1/3
    assert len(set(vals)) == len(vals)


# ------------------------------------------------------- supports and nesting
@pytest.mark.parametrize("n,levels", [(4, [1, 2]), (8, [0, 1, 2, 3]), (20, [1, 2, 4]), (30, [1, 2, 3, 6])])
def test_supports_are_nested_cyclic_windows(n, levels):
    pl = orc.plan(n, levels, SEED)
    prev = None
    for s, B in zip(levels, pl["B"]):
        supp = [set(np.nonzero(B[i])[0]) for i in range(n)]
        for i in range(n):
            # Definition 1: row weight (k/n)(sigma+1) with k = n; Lemma 1: cyclic window from i
            assert supp[i] == {(i + t) % n for t in range(s + 1)}
            assert B[i, i] == 1.0
        # every partition replicated sigma+1 times (Section II-C, minimum redundancy s+1)
        assert all(int((B[:, j] != 0).sum()) == s + 1 for j in range(n))
        if prev is not None:                      # Definition 2, second item
            assert all(prev[i] <= supp[i] for i in range(n))
        prev = supp
    # schedule: widest window left to right; level l done after s_l+1 tasks
    assert pl["schedule"].shape == (n, levels[-1] + 1)
    for i in range(n):
        assert list(pl["schedule"][i]) == [(i + t) % n for t in range(levels[-1] + 1)]
    assert list(pl["tasks_per_level"]) == [s + 1 for s in levels]


def test_sigma_zero_is_identity_and_all_ones_decoder():
    # Algorithm 1 initialisation: B_0 = I, A_0 = 1
    B = orc.coefficients(8, 0, SEED)
    assert np.array_equal(B, np.eye(8))
    a = orc.decode_vector(B, range(8))
    assert np.allclose(a, np.ones(8), atol=1e-14)


# --------------------------------------------------- Definition 1 brute force
def _exact_decoder(B, S):
    """Exact rational solve of a_S B_S = 1 by Gauss-Jordan over Fractions (test-side, independent)."""
    n = B.shape[0]
    S = list(S)
    m = len(S)
    rows = [[Fraction(B[S[c], j]) for c in range(m)] + [Fraction(1)] for j in range(n)]
    piv_rows = []
    r0 = 0
    for c in range(m):
        p = next((r for r in range(r0, n) if rows[r][c] != 0), None)
        assert p is not None, "rank deficient"
        rows[r0], rows[p] = rows[p], rows[r0]
        inv = 1 / rows[r0][c]
        rows[r0] = [v * inv for v in rows[r0]]
        for r in range(n):
            if r != r0 and rows[r][c] != 0:
                f = rows[r][c]
                rows[r] = [a - f * b for a, b in zip(rows[r], rows[r0])]
        piv_rows.append(r0)
        r0 += 1
    return [rows[r][m] for r in range(m)], rows[m:]


@pytest.mark.parametrize("n,levels", [(4, [1, 2]), (6, [1, 2, 3]), (8, [0, 1, 2, 3])])
def test_definition1_on_every_straggler_subset(n, levels):
    pl = orc.plan(n, levels, SEED)
    for s, B in zip(levels, pl["B"]):
        assert np.linalg.matrix_rank(B) == n - s
        for stragglers in itertools.combinations(range(n), s):
            S = [i for i in range(n) if i not in stragglers]
            BS = B[S]
            # every n-sigma rows span an (n-sigma)-dimensional space containing the all-ones vector
            sv = np.linalg.svd(BS, compute_uv=False)
            assert sv[-1] > 1e-9 * sv[0]
            assert np.linalg.matrix_rank(np.vstack([BS, np.ones(n)])) == n - s
            a = orc.decode_vector(B, S)
            assert set(np.nonzero(a)[0]) <= set(S)
            assert np.max(np.abs(a @ B - 1.0)) < 1e-9
            # unique solution: compare with an exact rational solve of the same fp64 matrix
            if n <= 6:
                exact, _ = _exact_decoder(B, S)
                assert np.allclose(a[S], [float(v) for v in exact], rtol=1e-8, atol=1e-10)


@pytest.mark.parametrize("n,levels,seed", [(20, [1, 2, 4], SEED + 1), (50, [1, 3, 5, 10], SEED + 2),
                                           (100, [1, 2, 5, 10], SEED + 3), (30, [1, 2, 3, 6], SEED + 4)])
def test_definition1_on_sampled_subsets_large_n(n, levels, seed):
    pl = orc.plan(n, levels, seed)
    rng = np.random.default_rng(7)
    for s, B in zip(levels, pl["B"]):
        # rows lie in an (n-s)-dim space containing 1: rank via SVD
        sv = np.linalg.svd(B, compute_uv=False)
        assert sv[n - s - 1] > 1e-8 * sv[0] and sv[n - s:].max(initial=0.0) < 1e-9 * sv[0]
        for _ in range(6):
            stragglers = rng.choice(n, size=s, replace=False)
            S = sorted(set(range(n)) - set(int(v) for v in stragglers))
            a = orc.decode_vector(B, S)
            assert np.max(np.abs(a @ B - 1.0)) < 1e-7 * max(1.0, np.abs(a).sum())
        # contiguous straggler blocks are the hardest windows for a cyclic code
        S = list(range(s, n))
        a = orc.decode_vector(B, S)
        assert np.max(np.abs(a @ B - 1.0)) < 1e-7 * max(1.0, np.abs(a).sum())


def test_rows_of_B_are_annihilated_by_zero_sum_matrix():
    # the all-ones vector and every row of B lie in one (n-sigma)-dim null space
    n, s = 12, 3
    B = orc.coefficients(n, s, SEED)
    # null space of B's row space complement: any vector orthogonal to rowspace(B) must sum to zero
    _, sv, Vt = np.linalg.svd(B)
    null = Vt[n - s:]                      # spans rowspace(B)^perp
    assert np.max(np.abs(null @ np.ones(n))) < 1e-10


def test_gepp_against_library_solver():
    rng = np.random.default_rng(3)
    for s in (1, 2, 5, 10):
        M = rng.uniform(-1, 1, size=(s, s))
        b = rng.uniform(-1, 1, size=s)
        assert np.allclose(orc._solve_gepp(M, b), np.linalg.solve(M, b), rtol=1e-9, atol=1e-12)
    # a system that NEEDS pivoting (zero leading entry)
    M = np.array([[0.0, 2.0], [1.0, 1.0]])
    assert np.allclose(orc._solve_gepp(M, np.array([2.0, 2.0])), [1.0, 1.0])


# ------------------------------------------------------- partial gradients
def _loss(kind, X, y, theta, hidden=0, C=0):
    X = np.asarray(X, dtype=np.float64)
    if kind == "lsq":
        return 0.5 * np.sum((X @ theta - y) ** 2)
    if kind == "logistic":
        z = X @ theta
        return np.sum(np.logaddexp(0.0, z) - y * z)
    if kind == "softmax":
        Z = X @ theta.reshape(X.shape[1], C)
        return np.sum(scipy.special.logsumexp(Z, axis=1) - Z[np.arange(len(y)), y])
    d = X.shape[1]
    W1 = theta[: d * hidden].reshape(d, hidden)
    b1 = theta[d * hidden: d * hidden + hidden]
    o = d * hidden + hidden
    W2 = theta[o: o + hidden * C].reshape(hidden, C)
    b2 = theta[o + hidden * C:]
    Z = np.maximum(X @ W1 + b1, 0) @ W2 + b2
    return np.sum(scipy.special.logsumexp(Z, axis=1) - Z[np.arange(len(y)), y])


@pytest.mark.parametrize("kind", ["lsq", "logistic", "softmax", "mlp"])
def test_gradients_by_finite_differences(kind):
    import scipy.special  # noqa: F401
    rng = np.random.default_rng(11)
    rows, d, hidden, C = 9, 5, 4, 3
    X = rng.normal(size=(rows, d))
    if kind == "lsq":
        y, theta = rng.normal(size=rows), rng.normal(size=d)
    elif kind == "logistic":
        y, theta = (rng.random(rows) < 0.5).astype(float), rng.normal(size=d)
    elif kind == "softmax":
        y, theta = rng.integers(0, C, rows), rng.normal(size=d * C)
    else:
        y, theta = rng.integers(0, C, rows), rng.normal(size=d * hidden + hidden + hidden * C + C)
    g = orc.partial_gradient(kind, X, y, theta, hidden, C)
    num = np.zeros_like(theta)
    h = 1e-6
    for p in range(theta.size):
        e = np.zeros_like(theta); e[p] = h
        num[p] = (_loss(kind, X, y, theta + e, hidden, C) - _loss(kind, X, y, theta - e, hidden, C)) / (2 * h)
    assert np.allclose(g, num, rtol=1e-5, atol=1e-6)


def test_lsq_gradient_vanishes_at_normal_equations():
    rng = np.random.default_rng(5)
    X, y = rng.normal(size=(40, 6)), rng.normal(size=40)
    theta = np.linalg.lstsq(X, y, rcond=None)[0]
    assert np.max(np.abs(orc.grad_lsq(X, y, theta))) < 1e-10


@pytest.mark.parametrize("kind", ["softmax", "mlp", "logistic"])
def test_gradients_against_autograd(kind):
    torch.manual_seed(0)
    rows, d, hidden, C = 33, 12, 16, 7
    X = torch.randn(rows, d, dtype=torch.float64)
    if kind == "logistic":
        y = (torch.rand(rows) < 0.5).double()
        th = torch.randn(d, dtype=torch.float64, requires_grad=True)
        loss = torch.nn.functional.binary_cross_entropy_with_logits(X @ th, y, reduction="sum")
        ynp = y.numpy()
    elif kind == "softmax":
        y = torch.randint(0, C, (rows,))
        th = torch.randn(d * C, dtype=torch.float64, requires_grad=True)
        loss = torch.nn.functional.cross_entropy(X @ th.view(d, C), y, reduction="sum")
        ynp = y.numpy()
    else:
        y = torch.randint(0, C, (rows,))
        th = torch.randn(d * hidden + hidden + hidden * C + C, dtype=torch.float64, requires_grad=True)
        W1 = th[: d * hidden].view(d, hidden)
        b1 = th[d * hidden: d * hidden + hidden]
        o = d * hidden + hidden
        W2 = th[o: o + hidden * C].view(hidden, C)
        b2 = th[o + hidden * C:]
        loss = torch.nn.functional.cross_entropy(torch.relu(X @ W1 + b1) @ W2 + b2, y, reduction="sum")
        ynp = y.numpy()
    loss.backward()
    g = orc.partial_gradient(kind, X.numpy(), ynp, th.detach().numpy(), hidden, C)
    assert np.allclose(g, th.grad.numpy(), rtol=1e-10, atol=1e-11)


def test_mlp_relu_mask_argument():
    # The optional ReLU decision: handing in the oracle's own decision (pre > 0) changes nothing, bit for bit ...
    rng = np.random.default_rng(3)
    rows, d, hidden, C = 17, 6, 5, 4
    X = rng.normal(size=(rows, d))
    y = rng.integers(0, C, rows)
    theta = rng.normal(size=d * hidden + hidden + hidden * C + C)
    W1 = theta[: d * hidden].reshape(d, hidden)
    b1 = theta[d * hidden: d * hidden + hidden]
    own = (X @ W1 + b1) > 0.0
    g0 = orc.grad_mlp(X, y, theta, hidden, C)
    assert np.array_equal(orc.grad_mlp(X, y, theta, hidden, C, relu_mask=own), g0)
    assert np.array_equal(orc.grad_mlp(X, y, theta, hidden, C, relu_mask=own.astype(np.int8)), g0)
    # ... an all-ones mask is the gradient of the network with the ReLU derivative replaced by 1 in the backward
    # pass only: dW2, db2 (which never see the mask) stay, dW1 = X^T (delta2 W2^T) by hand
    o = d * hidden + hidden
    W2 = theta[o: o + hidden * C].reshape(hidden, C)
    Z = np.maximum(X @ W1 + b1, 0) @ W2 + theta[o + hidden * C:]
    P = np.exp(Z - scipy.special.logsumexp(Z, axis=1, keepdims=True))
    P[np.arange(rows), y] -= 1.0
    g1 = orc.grad_mlp(X, y, theta, hidden, C, relu_mask=np.ones((rows, hidden)))
    assert np.allclose(g1[: d * hidden].reshape(d, hidden), X.T @ (P @ W2.T), rtol=1e-12, atol=1e-13)
    assert np.allclose(g1[d * hidden: o], (P @ W2.T).sum(axis=0), rtol=1e-12, atol=1e-13)
    assert np.array_equal(g1[o:], g0[o:])


def test_mlp_relu_mask_hand_case_one_flipped_unit():
    # 2 samples, 2 inputs, 2 hidden units, 2 classes, everything small enough to do by hand.
    # W1 = I, b1 = 0, so pre = X; sample 0 = (1, -1): unit 1 is off; sample 1 = (2, 3): both on.
    # W2 = [[1, 0], [0, 1]], b2 = 0.  Flipping the decision of (sample 0, unit 1) to "on" must add
    # x_0 * (delta2_0 . W2[1]) to column 1 of dW1 and delta2_0 . W2[1] to db1[1], and touch nothing else.
    X = np.array([[1.0, -1.0], [2.0, 3.0]])
    y = np.array([0, 1])
    theta = np.concatenate([np.eye(2).reshape(-1), np.zeros(2), np.eye(2).reshape(-1), np.zeros(2)])
    base = orc.grad_mlp(X, y, theta, 2, 2)
    mask = np.array([[1, 1], [1, 1]])                      # the oracle's own decision is [[1, 0], [1, 1]]
    flipped = orc.grad_mlp(X, y, theta, 2, 2, relu_mask=mask)
    # delta2 of sample 0 by hand: h = (1, 0), z = (1, 0), softmax = (e, 1) / (e + 1), label 0
    p1 = 1.0 / (math.e + 1.0)
    delta2_0 = np.array([-p1, p1])
    extra = delta2_0[1]                                    # delta2_0 . W2[1] with W2 = I
    diff = flipped - base
    want = np.zeros_like(base)
    want[0 * 2 + 1] = X[0, 0] * extra                      # dW1[0, 1]
    want[1 * 2 + 1] = X[0, 1] * extra                      # dW1[1, 1]
    want[4 + 1] = extra                                    # db1[1]
    assert np.allclose(diff, want, rtol=0, atol=1e-15)
    assert np.count_nonzero(diff) == 3


# ------------------------------------------- decoded gradient = full gradient
def _small_problem(kind, n, rows, d, hidden, C, seed):
    rng = np.random.default_rng(seed)
    X = rng.normal(size=(n, rows, d)) / math.sqrt(d)
    if kind == "lsq":
        y, theta = rng.normal(size=(n, rows)), rng.normal(size=d)
    elif kind == "logistic":
        y, theta = (rng.random((n, rows)) < 0.5).astype(float), rng.normal(size=d)
    elif kind == "softmax":
        y, theta = rng.integers(0, C, (n, rows)), rng.normal(size=d * C)
    else:
        y, theta = rng.integers(0, C, (n, rows)), rng.normal(size=d * hidden + hidden + hidden * C + C)
    return X, y, theta


@pytest.mark.parametrize("kind", ["lsq", "logistic", "softmax", "mlp"])
def test_decode_recovers_full_gradient_for_every_straggler_subset(kind):
    # Section II-C: the main node obtains the FULL gradient from any n - s responders
    n, levels, hidden, C = 5, [0, 1, 2], 6, 4
    X, y, theta = _small_problem(kind, n, 7, 6, hidden, C, 21)
    pl = orc.plan(n, levels, SEED)
    G = orc.partial_gradients(kind, X, y, theta, hidden, C)
    g_full = orc.full_gradient(kind, X, y, theta, hidden, C)
    assert np.allclose(G.sum(axis=0), g_full, rtol=1e-11, atol=1e-12)
    for s, B in zip(levels, pl["B"]):
        coded = orc.encode(B, G)
        for stragglers in itertools.combinations(range(n), s):
            S = [i for i in range(n) if i not in stragglers]
            a = orc.decode_vector(B, S)
            g = orc.decode(a, coded)
            assert np.linalg.norm(g - g_full) <= 1e-9 * np.linalg.norm(g_full)


def test_step_on_tiny_workload_brute_force():
    w = ngc_inputs.WORKLOADS["tiny"]
    X, y, theta = ngc_inputs.make_data(w)
    X, y, theta = X.numpy(), y.numpy(), theta.numpy()
    pl = orc.plan(w.n, list(w.levels), w.seed)
    g_full = orc.full_gradient("lsq", X, y, theta)
    n_tasks = w.levels[-1] + 1
    for size in range(0, 3):
        for stragglers in itertools.combinations(range(w.n), size):
            out = orc.step(pl, "lsq", X, y, theta, ngc_inputs.set_times(w.n, n_tasks, stragglers), 0.0, 0.0)
            want_level = 0 if size <= 1 else 1          # smallest listed tolerance that covers the set
            assert out["level"] == want_level
            assert not (set(out["S"]) & set(stragglers))
            assert len(out["S"]) == w.n - w.levels[want_level]
            assert np.linalg.norm(out["grad"] - g_full) <= 1e-9 * np.linalg.norm(g_full)
    # three stragglers exceed s_L = 2: never decodable
    assert orc.step(pl, "lsq", X, y, theta, ngc_inputs.set_times(w.n, n_tasks, [0, 1, 3]), 0.0, 0.0) is None


# ----------------------------------------------------------- selection rule
def test_selection_hand_cases():
    inf = np.inf
    # n = 4, levels {0,1}: level 0 needs all 4 workers' first task, level 1 needs 3 workers' two tasks
    t = np.array([[1.0, 1.0], [1.0, 1.0], [1.0, 1.0], [5.0, 1.0]])
    out = orc.select(t, [0, 1], 0.25, 0.125)
    assert out["level"] == 1 and list(out["S"]) == [0, 1, 2] and out["latency"] == 0.25 + 0.125 + 2.0
    assert list(out["tasks_done"]) == [2, 2, 2, 0]
    # level 0 wins when the slow worker is only slightly slow
    t[3, 0] = 1.5
    out = orc.select(t, [0, 1], 0.0, 0.0)
    assert out["level"] == 0 and list(out["S"]) == [0, 1, 2, 3] and out["latency"] == 1.5
    assert list(out["tasks_done"]) == [1, 1, 1, 1]
    # tie between levels -> smaller level index; tie between workers -> smaller worker index
    t = np.array([[1.0, 1.0], [1.0, 1.0], [1.0, 1.0], [2.0, 1.0]])
    out = orc.select(t, [0, 1], 0.0, 0.0)
    assert out["level"] == 0 and out["latency"] == 2.0
    t = np.ones((4, 2))
    out = orc.select(t, [1], 0.0, 0.0)
    assert list(out["S"]) == [0, 1, 2]
    # a dead worker: level 0 never decodable
    t = np.ones((4, 2)); t[2, :] = inf
    out = orc.select(t, [0, 1], 0.0, 0.0)
    assert out["level"] == 1 and list(out["S"]) == [0, 1, 3] and list(out["tasks_done"]) == [2, 2, 0, 2]
    t[0, :] = inf
    assert orc.select(t, [0, 1], 0.0, 0.0) is None


def test_observation1_load_matches_actual_straggler_count():
    # with s hard stragglers every responder computes at most the load of a GC with sigma = s
    n, levels = 8, [0, 1, 2, 3]
    for s in range(4):
        for stragglers in itertools.combinations(range(n), s):
            out = orc.select(ngc_inputs.set_times(n, 4, stragglers), levels, 0.0, 0.0)
            assert out["sigma"] == s
            assert out["tasks_done"].max() == s + 1
            assert all(out["tasks_done"][i] == 0 for i in stragglers)


def _mc_latencies(n, levels, lam, rho, gamma, eps, p_fail, trials, seed):
    rng = np.random.default_rng(seed)
    T = np.full(trials, np.inf)
    n_tasks = levels[-1] + 1
    for k in range(trials):
        t = rho + rng.exponential(1.0 / lam, size=(n, n_tasks))
        t[rng.random(n) < p_fail, :] = np.inf
        out = orc.select(t, levels, gamma, eps)
        if out is not None:
            T[k] = out["latency"]
    return T


def test_uncoded_ceiling_printed_in_section3():
    # Section III: n = 8, p_e = 0.05, sigma = 0: lim P(T <= t) ~ 0.66 = 0.95^8
    with open(os.path.join(GOLDEN, "paper_values.txt")) as f:
        vals = dict(line.split("#")[0].split() for line in f if line.strip() and not line.startswith("#"))
    printed = float(vals["uncoded_ceiling_n8_pe005"])
    assert abs(0.95 ** 8 - printed) < 0.005
    T = _mc_latencies(8, [0], 0.5, 0.5, 0.0, 0.1, 0.05, 20000, 1)
    frac = np.mean(np.isfinite(T))
    assert abs(frac - printed) < 0.012
    assert abs(latency.cdf_gc(1e6, 8, 0, 0.5, 0.5, 0.0, 0.1, 0.05) - 0.95 ** 8) < 1e-12


@pytest.mark.parametrize("sigma", [0, 1, 3])
def test_selection_matches_lemma2(sigma):
    n, lam, rho, gamma, eps, pe = 8, 0.5, 0.5, 0.3, 0.1, 0.05
    T = _mc_latencies(n, [sigma], lam, rho, gamma, eps, pe, 20000, 100 + sigma)
    for t in (3.0, 5.0, 8.0, 12.0, 18.0):
        want = latency.cdf_gc(t, n, sigma, lam, rho, gamma, eps, pe)
        assert abs(np.mean(T <= t) - want) < 0.015, (t, np.mean(T <= t), want)


@pytest.mark.parametrize("s_max", [1, 2, 3])
def test_selection_matches_theorem1(s_max):
    n, lam, rho, gamma, eps, pe = 8, 0.5, 0.5, 0.0, 0.1, 0.05
    T = _mc_latencies(n, list(range(s_max + 1)), lam, rho, gamma, eps, pe, 20000, 200 + s_max)
    for t in (3.0, 4.0, 6.0, 9.0, 14.0):
        want = latency.cdf_ngc(t, n, s_max, lam, rho, gamma, eps, pe)
        assert abs(np.mean(T <= t) - want) < 0.015, (t, np.mean(T <= t), want)


def test_theorem1_reduces_to_lemma2_and_ceilings():
    # s_max = 0: the nested code IS the uncoded scheme
    for t in (2.0, 4.0, 9.0):
        assert abs(latency.cdf_ngc(t, 8, 0, 0.5, 0.5, 0.0, 0.1, 0.05)
                   - latency.cdf_gc(t, 8, 0, 0.5, 0.5, 0.0, 0.1, 0.05)) < 1e-12
    # ceilings: outer sums of Lemma 2 / Theorem 1 = binomial CDF of the number of failed workers
    for s in range(5):
        want = scipy.stats.binom.cdf(s, 8, 0.05)
        assert abs(latency.cdf_ngc(1e6, 8, s, 0.5, 0.5, 0.0, 0.1, 0.05) - want) < 1e-10
        assert abs(latency.cdf_gc(1e6, 8, s, 0.5, 0.5, 0.0, 0.1, 0.05) - want) < 1e-10
    # the nested code is never slower than the fixed code of the same tolerance (Section IV discussion)
    for t in np.linspace(2.0, 18.0, 17):
        assert latency.cdf_ngc(t, 8, 3, 0.5, 0.5, 0.0, 0.1, 0.05) >= latency.cdf_gc(t, 8, 3, 0.5, 0.5, 0.0, 0.1, 0.05) - 1e-12


def test_erlang_reading_of_eq3():
    lam = 0.7
    for u in (1, 2, 4):
        for t in (0.5, 2.0, 6.0):
            # library Erlang CDF, shift gamma + eps + u rho
            want = scipy.stats.gamma.cdf(t - (0.2 + 0.1 + u * 0.5), a=u, scale=1.0 / lam)
            assert abs(latency.cdf_tasks(u, t, lam, 0.5, 0.2, 0.1) - want) < 1e-12
            # identity in the proof of Corollary 1 (rho = 0)
            diff = latency.cdf_tasks(u, t, lam, 0.0, 0.0, 0.0) - latency.cdf_tasks(u + 1, t, lam, 0.0, 0.0, 0.0)
            assert abs(diff - math.exp(-lam * t) * (lam * t) ** u / math.factorial(u)) < 1e-12


# ------------------------------------- the oracle's own task-time sampler (Section II-D)
def test_oracle_trial_seed_is_the_published_stream():
    # trial r of a run uses output r + 1 of the SplitMix64 stream seeded with (seed xor a fixed constant):
    # with the seed chosen so that the xor gives 1234567, the published vector of the generator must come out
    seed = 1234567 ^ 0xD1B54A32D192ED03
    assert latency.trial_seed(seed, 0) == 6457827717110365317
    assert latency.trial_seed(seed, 1) == 3203168211198807973
    assert latency.trial_seed(seed, 4) == 16408922859458223821


def test_oracle_sampler_follows_the_response_time_model():
    # Section II-D: a task takes rho + Exp(lambda); a worker fails, with all its tasks, with probability p_e
    n, tasks, rho, lam, pe = 4000, 5, 0.5, 2.0, 0.2
    t = np.array(latency.sample_times(99, n, tasks, rho, lam, pe))
    dead = np.isinf(t[:, 0])
    assert all(np.isinf(t[i]).all() if dead[i] else np.isfinite(t[i]).all() for i in range(n))
    assert abs(dead.mean() - pe) < 4 * math.sqrt(pe * (1 - pe) / n)
    x = t[~dead].reshape(-1) - rho
    assert x.min() > 0.0
    m = x.size
    assert abs(x.mean() - 1 / lam) < 5 / lam / math.sqrt(m)
    assert abs(x.var() - 1 / lam ** 2) < 0.05 / lam ** 2
    assert scipy.stats.kstest(x, "expon", args=(0, 1 / lam)).pvalue > 1e-3
    # tasks of one worker and of different workers are not copies of each other
    assert len(np.unique(x)) == m
    # the first uniform of the stream, by hand: position 2 of seed 1234567 is 3203168211198807973
    u = ((3203168211198807973 >> 11) + 0.5) / 2.0 ** 53
    one = latency.sample_times(1234567, 1, 1, 0.25, 4.0, 0.0)[0][0]
    assert abs(one - (0.25 - math.log(u) / 4.0)) < 1e-15


@pytest.mark.parametrize("sigma", [0, 2])
def test_lemma2_on_the_oracle_sampler(sigma):
    # the same Monte Carlo as above, with the task times drawn by the oracle's SplitMix64 sampler
    n, lam, rho, gamma, eps, pe, trials = 8, 0.5, 0.5, 0.3, 0.1, 0.05, 6000
    T = np.full(trials, np.inf)
    for r in range(trials):
        t = np.array(latency.sample_times(latency.trial_seed(4242 + sigma, r), n, sigma + 1, rho, lam, pe))
        out = orc.select(t, [sigma], gamma, eps)
        if out is not None:
            T[r] = out["latency"]
    for t in (3.0, 5.0, 8.0, 12.0, 18.0):
        want = latency.cdf_gc(t, n, sigma, lam, rho, gamma, eps, pe)
        assert abs(np.mean(T <= t) - want) < 0.025, (t, np.mean(T <= t), want)


# ----------------------------------------------------- stored oracle outputs
def test_stored_tiny_B_is_reproduced():
    # regression guard: values written by tests/golden/make_golden.py (calls only the oracle)
    stored = np.loadtxt(os.path.join(GOLDEN, "B_tiny_oracle.txt"), dtype=str)
    w = ngc_inputs.WORKLOADS["tiny"]
    pl = orc.plan(w.n, list(w.levels), w.seed)
    got = np.concatenate([B.reshape(-1) for B in pl["B"]])
    assert [float.fromhex(v) for v in stored] == list(got)
