"""Failure reporting and ordering of the GPU entry points, without making anything fail on the GPU.

* a bounded device-side wait that runs out (a barrier nobody completes: nothing faults, nothing hangs) must end in
  NGC_ERR_TIMEOUT from ngc_device_status, once, and leave the plan and the context usable;
* a replayed CUDA graph of ngc_step followed, with no synchronisation, by an eager ngc_step with another
  responsive set: the eager step's decoding-vector solve (on the plan's side stream) must not overwrite the
  vector while the replayed decode still reads it.
"""
import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import coded_torch_dtype, model_of, rel_l2, to_np64

pytestmark = pytest.mark.gpu

NGC_ERR_TIMEOUT = -5


def _small(name, rows):
    from dataclasses import replace
    return replace(ngc_inputs.shrink(ngc_inputs.WORKLOADS[name], rows=rows), pattern="sets")


def test_a_wait_that_runs_out_is_reported_and_the_plan_stays_usable():
    w = _small("logistic20", 64)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    l = w.n_params
    coded = torch.empty((w.n, l), dtype=coded_torch_dtype(p.coded_dtype(m)), device="cuda")
    grad = torch.empty(l, dtype=torch.float32, device="cuda")
    t = ngc_inputs.set_times(w.n, w.levels[-1] + 1, [3])
    g_full = orc.full_gradient(w.kind, to_np64(X), to_np64(y), to_np64(theta))
    p.step(m, theta, X, y, t, coded, grad)
    assert p.device_status_code() == 0
    # one warp waits 100 000 cycles (~50 us) on a barrier without arrivals, gives up, sets the status word
    p.selftest_wait_timeout(100_000)
    assert p.device_status_code() == NGC_ERR_TIMEOUT
    assert p.device_status_code() == 0                      # reported once
    with pytest.raises(ngc.NgcError):
        p.selftest_wait_timeout(0)
    # the context and the plan are intact
    grad.zero_()
    p.step(m, theta, X, y, t, coded, grad)
    torch.cuda.synchronize()
    assert p.device_status_code() == 0
    assert rel_l2(grad.cpu().numpy(), g_full) < 1e-5


@pytest.mark.parametrize("name,rows,tol", [("logistic20", 256, 1e-5), ("softmax50", 256, 1e-2)])
def test_eager_step_right_after_a_graph_replay_does_not_disturb_the_replayed_decode(name, rows, tol):
    w = _small(name, rows)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    l = w.n_params
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    cdt = coded_torch_dtype(p.coded_dtype(m))
    coded_a = torch.empty((w.n, l), dtype=cdt, device="cuda")
    coded_b = torch.empty((w.n, l), dtype=cdt, device="cuda")
    grad_a = torch.zeros(l, dtype=torch.float32, device="cuda")
    grad_b = torch.zeros(l, dtype=torch.float32, device="cuda")
    n_tasks = w.levels[-1] + 1
    t_a = ngc_inputs.set_times(w.n, n_tasks, [0])                       # first level, worker 0 missing
    t_b = ngc_inputs.set_times(w.n, n_tasks, list(range(1, 1 + w.levels[-1])))   # last level, other workers missing
    p.step(m, theta, X, y, t_a, coded_a, grad_a)                        # eager once: allocates, creates the side stream
    p.step(m, theta, X, y, t_b, coded_b, grad_b)
    torch.cuda.synchronize()
    want_a, want_b = grad_a.clone(), grad_b.clone()
    g_full = orc.full_gradient(w.kind, to_np64(X), to_np64(y), to_np64(theta), w.hidden, w.n_classes)
    assert rel_l2(want_a.cpu().numpy(), g_full) < tol and rel_l2(want_b.cpu().numpy(), g_full) < tol

    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        p.step(m, theta, X, y, t_a, coded_a, grad_a, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    graph.replay()                                                      # on its own: the captured step's result
    torch.cuda.synchronize()
    assert rel_l2(grad_a.cpu().numpy(), want_a.cpu().numpy()) < 1e-6    # (in-order decode: other summation order)
    want_a = grad_a.clone()
    for _ in range(20):
        grad_a.zero_()
        grad_b.zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            graph.replay()                                              # captured step: in-order solve + decode
            p.step(m, theta, X, y, t_b, coded_b, grad_b, stream.cuda_stream)   # eager: solve on the side stream
        torch.cuda.synchronize()
        assert torch.equal(grad_a, want_a)
        assert torch.equal(grad_b, want_b)
    assert p.device_status_code() == 0
