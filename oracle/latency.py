"""Closed-form latency CDFs of Section IV -- TEST INFRASTRUCTURE ONLY.

Used to pin the oracle's stopping rule by Monte Carlo: the empirical CDF of
the latency that `ngc_oracle.select` reports for sampled task times must
match Lemma 2 (one component code) and Theorem 1 (nested code).

Pin status: the closed forms against scipy's gamma / binomial distributions, the identity in the
proof of Corollary 1, the printed 0.66 ceiling and Monte Carlo of the selection rule; the task-time
sampler against the published SplitMix64 vector (trial seeds, one draw worked by hand), the moments
and a Kolmogorov-Smirnov test of the shifted exponential, the failure rate, and Lemma 2 by Monte
Carlo on its own draws.
"""
from __future__ import annotations

from math import comb, exp, factorial, inf, log

from .ngc_oracle import splitmix64_at


def cdf_tasks(u: int, t: float, lam: float, rho: float, gamma: float, eps: float) -> float:
    """F_u(t) = P(T_i^(u) <= t), Eq. 3: shift gamma + eps + u*rho plus Erlang(u, lam).

    Eq. 3 prints the sum up to k = u; an Erlang of shape u has terms
    k = 0..u-1, and only that reading gives F_u - F_{u+1} = e^{-lam t}(lam t)^u / u!
    at rho = 0, the identity used in the proof of Corollary 1.
    """
    if u == 0:
        return 1.0
    x = t - (gamma + eps + u * rho)
    if x <= 0.0:
        return 0.0
    tail = 0.0
    for k in range(u):
        tail += (lam * x) ** k / factorial(k)
    return 1.0 - tail * exp(-lam * x)


def cdf_gc(t, n, sigma, lam, rho, gamma, eps, p_fail) -> float:
    """Lemma 2: latency CDF of an (n, k, sigma) gradient code."""
    F = cdf_tasks(sigma + 1, t, lam, rho, gamma, eps)
    total = 0.0
    for kappa in range(sigma + 1):
        alive = n - kappa
        cond = 0.0
        for tau in range(n - sigma, alive + 1):
            cond += comb(alive, tau) * F ** tau * (1.0 - F) ** (alive - tau)
        total += cond * comb(n, kappa) * p_fail ** kappa * (1.0 - p_fail) ** (n - kappa)
    return total


def cdf_ngc(t, n, s_max, lam, rho, gamma, eps, p_fail) -> float:
    """Theorem 1: latency CDF of an (n, k, s_max) nested gradient code.

    Given kappa failed workers, every alive worker has independently finished
    exactly u tasks (u = 0..s_max) or at least s_max + 1 by time t.  The main
    node cannot decode iff for every u = 1..s_max+1 at most n - u workers
    have finished u or more tasks.  The proof states this cumulative
    condition; the printed summation limit drops the running sum from its
    first argument, so the proof's sentence is followed.
    """
    F = [cdf_tasks(u, t, lam, rho, gamma, eps) for u in range(s_max + 3)]
    q = [F[u] - F[u + 1] for u in range(s_max + 1)] + [F[s_max + 1]]   # q[u], u = 0..s_max+1

    def not_decodable(u: int, used: int, alive: int) -> float:
        # sum over i_u given that `used` workers have finished more than u tasks
        if u == 0:
            return q[0] ** (alive - used)
        limit = min(n - u - used, alive - used)
        acc = 0.0
        for i_u in range(0, limit + 1):
            acc += comb(alive - used, i_u) * q[u] ** i_u * not_decodable(u - 1, used + i_u, alive)
        return acc

    total = 0.0
    for kappa in range(s_max + 1):
        alive = n - kappa
        cond = 1.0 - not_decodable(s_max + 1, 0, alive)
        total += cond * comb(n, kappa) * p_fail ** kappa * (1.0 - p_fail) ** (n - kappa)
    return total


def sample_times(seed: int, n: int, tasks: int, shift: float, rate: float, p_fail: float):
    """Response-time model of Section II-D from the SplitMix64 stream: worker i is dead when the uniform at
    position 1 + i (tasks+1) is below p_fail; its m-th task takes shift - log(u) / rate with u the uniform
    (bits + 1/2) / 2^53 at position 2 + i (tasks+1) + m."""
    out = []
    for i in range(n):
        base = i * (tasks + 1)
        dead = (splitmix64_at(seed, 1 + base) >> 11) / 9007199254740992.0 < p_fail
        row = []
        for m in range(tasks):
            u = ((splitmix64_at(seed, 2 + base + m) >> 11) + 0.5) / 9007199254740992.0
            row.append(inf if dead else shift - log(u) / rate)
        out.append(row)
    return out


def trial_seed(seed: int, trial: int) -> int:
    """Seed of Monte-Carlo trial `trial` of a run seeded with `seed`."""
    return splitmix64_at(seed ^ 0xD1B54A32D192ED03, trial + 1)
