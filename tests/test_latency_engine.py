"""Latency engine (Section IV): closed forms of the library against the oracle's, the SplitMix64 sampler on
both sides, and the GPU Monte Carlo of the stopping rule against the oracle trial by trial and against
Theorem 1 / Lemma 2 in distribution."""
import numpy as np
import pytest
import torch

import paper_2212_08580_b200 as ngc
from oracle import latency as olat
from oracle import ngc_oracle as orc

PAPER = dict(lam=0.5, rho=0.5, eps=0.1, p_fail=0.05)   # parameters of the paper's figures (n = k = 8)


def test_closed_forms_match_oracle():
    for t in np.linspace(1.0, 20.0, 39):
        for s in range(0, 7):
            a = ngc.latency_cdf_gc(8, s, t, PAPER["lam"], PAPER["rho"], 0.25, PAPER["eps"], PAPER["p_fail"])
            b = olat.cdf_gc(t, 8, s, PAPER["lam"], PAPER["rho"], 0.25, PAPER["eps"], PAPER["p_fail"])
            assert abs(a - b) < 1e-12
            a = ngc.latency_cdf_ngc(8, s, t, PAPER["lam"], PAPER["rho"], 0.25, PAPER["eps"], PAPER["p_fail"])
            b = olat.cdf_ngc(t, 8, s, PAPER["lam"], PAPER["rho"], 0.25, PAPER["eps"], PAPER["p_fail"])
            assert abs(a - b) < 1e-12
    assert abs(ngc.latency_cdf_gc(8, 0, 1e6, 0.5, 0.5, 0.0, 0.1, 0.05) - 0.95 ** 8) < 1e-12   # Section III: ~0.66
    assert ngc.latency_cdf_ngc(8, 9, 1.0, 0.5, 0.5, 0.0, 0.1, 0.05) < 0                         # s_max >= n: refused
    # the nested code dominates the fixed code of the same tolerance; larger s_max never hurts (Section IV)
    for t in np.linspace(2.0, 18.0, 17):
        v = [ngc.latency_cdf_ngc(8, s, t, 0.5, 0.5, 0.0, 0.1, 0.05) for s in (2, 4, 6)]
        assert v[0] <= v[1] + 1e-12 <= v[2] + 2e-12
        assert ngc.latency_cdf_ngc(8, 3, t, 0.5, 0.5, 0.0, 0.1, 0.05) >= ngc.latency_cdf_gc(8, 3, t, 0.5, 0.5, 0.0, 0.1, 0.05) - 1e-12


def test_sampler_matches_oracle_sampler():
    got = ngc.sample_times(77, 30, 7, 0.5, 2.0, 0.2)
    want = np.array(olat.sample_times(77, 30, 7, 0.5, 2.0, 0.2))
    assert np.array_equal(np.isinf(got), np.isinf(want)) and np.isinf(want).any()
    fin = np.isfinite(want)
    assert np.allclose(got[fin], want[fin], rtol=1e-14, atol=0)


@pytest.mark.gpu
@pytest.mark.parametrize("n,levels", [(8, [0, 1, 2, 3]), (20, [1, 2, 4]), (100, [1, 2, 5, 10])])
def test_monte_carlo_trials_match_oracle(n, levels):
    gamma, eps, rho, lam, pf = 0.3, 0.1, 0.5, 0.5, 0.05
    p = ngc.Plan(n, levels, seed=1, gamma=gamma, eps=eps)
    trials = 400
    lat = torch.empty(trials, dtype=torch.float64, device="cuda")
    lev = torch.empty(trials, dtype=torch.int32, device="cuda")
    p.latency_mc(2024, rho, lam, pf, lat, lev)
    torch.cuda.synchronize()
    lat, lev = lat.cpu().numpy(), lev.cpu().numpy()
    mism = 0
    for r in range(trials):
        t = np.array(olat.sample_times(olat.trial_seed(2024, r), n, levels[-1] + 1, rho, lam, pf))
        want = orc.select(t, levels, gamma, eps)
        if want is None:
            assert lev[r] == -1 and np.isinf(lat[r])
            continue
        assert abs(lat[r] - want["latency"]) <= 1e-12 * want["latency"]
        mism += int(lev[r] != want["level"])          # only a tie within rounding can differ
    assert mism == 0


@pytest.mark.gpu
def test_monte_carlo_reproduces_theorem1_and_lemma2():
    trials = 400000
    lat = torch.empty(trials, dtype=torch.float64, device="cuda")
    lev = torch.empty(trials, dtype=torch.int32, device="cuda")
    grid = np.linspace(2.0, 18.0, 33)
    for s_max in (2, 3, 6):
        p = ngc.Plan(8, list(range(s_max + 1)), seed=1, gamma=0.0, eps=PAPER["eps"])
        p.latency_mc(11 + s_max, PAPER["rho"], PAPER["lam"], PAPER["p_fail"], lat, lev)
        torch.cuda.synchronize()
        T = lat.cpu().numpy()
        for t in grid:
            want = olat.cdf_ngc(t, 8, s_max, PAPER["lam"], PAPER["rho"], 0.0, PAPER["eps"], PAPER["p_fail"])
            assert abs(np.mean(T <= t) - want) < 0.004
    for sigma in (0, 3):
        p = ngc.Plan(8, [sigma], seed=1, gamma=0.0, eps=PAPER["eps"])
        p.latency_mc(21 + sigma, PAPER["rho"], PAPER["lam"], PAPER["p_fail"], lat, lev)
        torch.cuda.synchronize()
        T = lat.cpu().numpy()
        for t in grid:
            want = olat.cdf_gc(t, 8, sigma, PAPER["lam"], PAPER["rho"], 0.0, PAPER["eps"], PAPER["p_fail"])
            assert abs(np.mean(T <= t) - want) < 0.004
        if sigma == 0:
            assert abs(np.mean(np.isfinite(T)) - 0.66) < 0.01     # the ceiling printed in Section III
