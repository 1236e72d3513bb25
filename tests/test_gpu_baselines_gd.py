"""The comparison schemes of the paper through the same library (a fixed gradient code and the uncoded scheme
are plans with a single level), their load accounting, and gradient descent (Eq. 1) driven by ngc_step."""
import itertools

import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import model_of, rel_l2, to_np64


def test_fixed_code_overhead_versus_nested_code():
    # Section III: with s < sigma actual stragglers a fixed (n, k, sigma) code makes every responder compute
    # sigma + 1 tasks, a factor (sigma+1)/(s+1) more than the nested code, which stops at the component s.
    n, sigma = 8, 3
    gc = ngc.Plan(n, [sigma], seed=1)
    nested = ngc.Plan(n, [0, 1, 2, 3], seed=1)
    for s in range(sigma + 1):
        for stragglers in itertools.combinations(range(n), s):
            t = ngc_inputs.set_times(n, sigma + 1, stragglers)
            a, b = gc.select(t), nested.select(t)
            assert a.sigma == sigma and a.nS == n - sigma              # sigma - s responders are ignored
            assert max(a.tasks_done[:n]) == sigma + 1
            assert b.sigma == s and max(b.tasks_done[:n]) == s + 1
            assert a.latency / b.latency == (sigma + 1) / (s + 1)       # unit task times: load ratio = time ratio
    # the uncoded scheme tolerates nothing
    unc = ngc.Plan(n, [0], seed=1)
    assert unc.select(ngc_inputs.set_times(n, 1, [])).nS == n
    with pytest.raises(ngc.NgcError):
        unc.select(ngc_inputs.set_times(n, 1, [2]))


@pytest.mark.gpu
@pytest.mark.parametrize("levels", [[0], [3]])
def test_single_level_plans_decode_the_full_gradient(levels):
    w = ngc_inputs.Workload("gc_case", 900, 8, tuple(levels), "logistic", 200, 512, "f32")
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    p = ngc.Plan(w.n, levels, seed=w.seed)
    g_full = orc.full_gradient("logistic", to_np64(X), to_np64(y), to_np64(theta))
    coded = torch.empty((w.n, w.d), dtype=torch.float64, device="cuda")
    grad = torch.empty(w.d, dtype=torch.float32, device="cuda")
    for stragglers in ([], list(range(levels[0]))):
        t = ngc_inputs.set_times(w.n, levels[0] + 1, stragglers)
        info = p.step(model_of(w), theta, X, y, t, coded, grad)
        torch.cuda.synchronize()
        assert info.sigma == levels[0]
        assert rel_l2(grad.cpu().numpy(), g_full) < 1e-5


@pytest.mark.gpu
def test_gradient_descent_follows_the_oracle():
    # Eq. 1: theta <- theta - (eta / m) g, g decoded under a fresh straggler pattern every iteration
    w = ngc_inputs.Workload("gd_case", 901, 6, (1, 2), "lsq", 300, 256, "f32", unit_x=True)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m_rows = w.n * w.rows
    eta = 0.5
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    pl = orc.plan(w.n, list(w.levels), w.seed)
    Xn, yn = to_np64(X), to_np64(y)
    th_o = to_np64(theta).copy()
    coded = torch.empty((w.n, w.d), dtype=torch.float64, device="cuda")
    grad = torch.empty(w.d, dtype=torch.float32, device="cuda")
    th = theta.clone()
    stream = torch.cuda.current_stream().cuda_stream
    losses = []
    for it in range(8):
        t = ngc_inputs.sample_times(w.n, w.levels[-1] + 1, 1234 + it)
        p.step(model_of(w), th, X, y, t, coded, grad, stream)
        ngc.gd_update(th, grad, eta / m_rows, stream)
        out = orc.step(pl, "lsq", Xn, yn, th_o, t, 0.0, 0.0)
        th_o = th_o - (eta / m_rows) * out["grad"]
        losses.append(0.5 * float(np.sum((Xn.reshape(-1, w.d) @ th_o - yn.reshape(-1)) ** 2)))
    torch.cuda.synchronize()
    assert rel_l2(th.cpu().numpy(), th_o) < 1e-5
    assert all(b < a for a, b in zip(losses, losses[1:]))      # the loss goes down every iteration


@pytest.mark.gpu
@pytest.mark.parametrize("name,rows,tol", [("logistic20", 128, 1e-5), ("mlp30", 200, 1e-2)])
def test_gradient_descent_iteration_replayed_from_a_cuda_graph(name, rows, tol):
    """One iteration (ngc_step for a fixed straggler pattern + the update of Eq. 1) captured into a CUDA graph
    and replayed: every replay must do what the eager calls do on the parameters as they then stand, and the
    plan must stay usable for eager steps afterwards."""
    from dataclasses import replace
    w = replace(ngc_inputs.shrink(ngc_inputs.WORKLOADS[name], rows=rows), pattern="sets")
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    l = w.n_params
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    cdt = p.coded_dtype(m)
    coded = torch.empty((w.n, l), dtype=torch.float64 if cdt == ngc.NGC_F64 else torch.float32, device="cuda")
    grad = torch.empty(l, dtype=torch.float32, device="cuda")
    t = ngc_inputs.set_times(w.n, w.levels[-1] + 1, [1, 4])
    eta = 1e-3 / (w.n * w.rows)

    def eager(th, steps):
        th = th.clone()
        for _ in range(steps):
            p.step(m, th, X, y, t, coded, grad)
            ngc.gd_update(th, grad, eta)
        torch.cuda.synchronize()
        return th

    want1, want3 = eager(theta, 1), eager(theta, 3)       # also allocates everything the plan needs
    th = theta.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        s = torch.cuda.current_stream().cuda_stream
        p.step(m, th, X, y, t, coded, grad, s)
        ngc.gd_update(th, grad, eta, s)
    torch.cuda.synchronize()
    assert torch.equal(th, theta)                         # capture runs nothing
    graph.replay()
    torch.cuda.synchronize()
    assert rel_l2(th.cpu().numpy(), want1.cpu().numpy()) < 1e-6
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert rel_l2(th.cpu().numpy(), want3.cpu().numpy()) < 1e-6
    # eager steps on the same plan still work, and decode the full gradient
    info = p.step(m, theta, X, y, t, coded, grad)
    torch.cuda.synchronize()
    g_full = orc.full_gradient(w.kind, to_np64(X), to_np64(y), to_np64(theta), w.hidden, w.n_classes)
    assert info.sigma == 2 and rel_l2(grad.cpu().numpy(), g_full) < tol
    assert p.device_status() < 1e-6


@pytest.mark.gpu
def test_nested_code_never_waits_longer_than_a_fixed_code_on_the_same_times():
    """Section III: with negligible signalling time a nested code with levels 0..s_bar stops, in every iteration,
    as early as the best fixed code does on the same task times, and its responders compute no more than that
    code's load; gradient descent ends at the same parameters whichever code decodes the gradients."""
    from paper_2212_08580_b200 import gd_loop
    n, s_bar, iters = 8, 3, 12
    w = ngc_inputs.Workload("gd_compare", 902, n, (0,), "lsq", 128, 128, "f32", unit_x=True)
    X, y, theta0 = ngc_inputs.make_data(w, "cuda")
    step = 0.5 / (n * w.rows)
    hist, finals = {}, {}
    for name, levels in [("nested", list(range(s_bar + 1)))] + [(s, [s]) for s in range(s_bar + 1)]:
        plan = ngc.Plan(n, levels, seed=5, gamma=0.0, eps=0.0)
        th = theta0.clone()
        hist[name] = gd_loop.run(plan, model_of(w), th, X, y, iters, step, seed=4242, rho=0.5, lam=0.5, p_fail=0.0,
                                 times_width=s_bar + 1)
        torch.cuda.synchronize()
        finals[name] = th.cpu().numpy()
    for it in range(iters):
        best = min(hist[s].latency[it] for s in range(s_bar + 1))
        assert hist["nested"].latency[it] == best                      # same times, same arithmetic: equal, not just close
        s_used = hist["nested"].level[it]                              # level index = tolerance for levels 0..s_bar
        assert hist[s_used].latency[it] == best
    assert hist["nested"].total_latency <= min(hist[s].total_latency for s in range(s_bar + 1))
    for s in range(s_bar + 1):
        assert rel_l2(finals[s], finals["nested"]) < 1e-5
