"""Steps queued back to back without a host synchronisation in between: every step must decode with the vector
of its own straggler pattern and level, although the decoding vectors of consecutive steps share one buffer and
are solved on a stream of their own."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import coded_torch_dtype, model_of, oracle_G, rel_l2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,rows,tol", [("logistic20", 192, 1e-5), ("lsq100", 96, 1e-5), ("softmax50", 256, 1e-2)])
def test_queued_steps_each_use_their_own_decoding_vector(name, rows, tol):
    # straggler sets of sweeping size, so that consecutive steps land on different levels
    w = replace(ngc_inputs.shrink(ngc_inputs.WORKLOADS[name], rows=rows), pattern="sets")
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    l = w.n_params
    coded = torch.empty((w.n, l), dtype=coded_torch_dtype(p.coded_dtype(m)), device="cuda")
    steps = 24
    grads = torch.zeros((steps, l), dtype=torch.float32, device="cuda")
    g_full = oracle_G(w, X, y, theta).sum(axis=0)
    ran, levels = [], set()
    for it in range(steps):
        t = ngc_inputs.pattern_times(w, it)
        want = orc.select(t, list(w.levels), 0.0, 0.0)
        if want is None:
            continue
        info = p.step(m, theta, X, y, t, coded, grads[it])      # no synchronisation here
        assert info.layer == want["level"] and np.array_equal(info.responsive(), want["S"])
        ran.append(it)
        levels.add(info.layer)
    torch.cuda.synchronize()
    assert len(ran) >= 16 and len(levels) >= 2                   # the vectors of consecutive steps really differ
    got = grads.cpu().numpy()
    for it in ran:
        assert rel_l2(got[it], g_full) < tol, it
    assert p.device_status() < 1e-6


@pytest.mark.parametrize("name,rows", [("softmax50", 300), ("mlp30", 200)])
def test_step_of_a_dense_model_matches_encode_then_decode(name, rows):
    """ngc_step lets the decode ride on the encode kernel of the dense models; ngc_grad_encode followed by
    ngc_decode reads the coded matrix back.  Same coded rows bit for bit, same decoded gradient up to the
    order of the fp64 sums."""
    w = replace(ngc_inputs.shrink(ngc_inputs.WORKLOADS[name], rows=rows), pattern="sets")
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    l = w.n_params
    cdt = p.coded_dtype(m)
    coded_a = torch.empty((w.n, l), dtype=coded_torch_dtype(cdt), device="cuda")
    coded_b = torch.empty_like(coded_a)
    grad_a = torch.empty(l, dtype=torch.float32, device="cuda")
    grad_b = torch.empty_like(grad_a)
    for it in (0, 3, 7, 10):                                      # straggler sets of different sizes: several levels
        t = ngc_inputs.pattern_times(w, it)
        coded_a.fill_(float("nan"))
        grad_a.fill_(float("nan"))
        info = p.step(m, theta, X, y, t, coded_a, grad_a)
        p.grad_encode(m, theta, X, y, info.layer, coded_b)
        p.decode(info.layer, info.responsive(), coded_b, cdt, l, grad_b)
        torch.cuda.synchronize()
        assert torch.equal(coded_a, coded_b)
        ga, gb = grad_a.cpu().numpy(), grad_b.cpu().numpy()
        assert np.isfinite(ga).all()
        assert rel_l2(ga, gb) < 1e-6, (it, info.layer, rel_l2(ga, gb))
    assert p.device_status() < 1e-6


def test_one_plan_serves_models_of_growing_and_changing_kind():
    """The plan's scratch grows with the model it is asked to serve and its choice of decode path follows the
    model: least squares, then a larger logistic model, softmax regression, an MLP, and least squares again."""
    n, levels = 6, (1, 2)
    p = ngc.Plan(n, levels, seed=77)
    cases = [
        ngc_inputs.Workload("mix_lsq", 950, n, levels, "lsq", 64, 128, "f32", pattern="sets", unit_x=True),
        ngc_inputs.Workload("mix_logistic", 951, n, levels, "logistic", 300, 2048, "f32", pattern="sets"),
        ngc_inputs.Workload("mix_softmax", 952, n, levels, "softmax", 300, 256, "bf16", n_classes=256, pattern="sets"),
        ngc_inputs.Workload("mix_mlp", 953, n, levels, "mlp", 260, 64, "f32", n_classes=10, hidden=128, pattern="sets"),
        ngc_inputs.Workload("mix_lsq", 950, n, levels, "lsq", 64, 128, "f32", pattern="sets", unit_x=True),
    ]
    seen = 0
    for it, w in enumerate(cases):
        X, y, theta = ngc_inputs.make_data(w, "cuda")
        m = model_of(w)
        l = w.n_params
        coded = torch.empty((n, l), dtype=coded_torch_dtype(p.coded_dtype(m)), device="cuda")
        grad = torch.empty(l, dtype=torch.float32, device="cuda")
        t = ngc_inputs.set_times(n, levels[-1] + 1, list(range(it % 3)))
        info = p.step(m, theta, X, y, t, coded, grad)             # queued behind the previous model's step
        torch.cuda.synchronize()
        g_full = oracle_G(w, X, y, theta).sum(axis=0)
        tol = 1e-5 if w.kind in ("lsq", "logistic") else 1e-2
        assert rel_l2(grad.cpu().numpy(), g_full) < tol, (w.name, info.layer)
        assert p.workspace_bytes() >= seen
        seen = p.workspace_bytes()
    assert p.device_status() < 1e-6


@pytest.mark.parametrize("name,rows", [("softmax50", 520), ("mlp30", 2000)])
def test_dense_steps_are_bitwise_reproducible(name, rows):
    """Nothing in the dense paths is added up in an order that depends on timing: per-CTA slots and worker
    chunks are summed in index order.  mlp30 at its full row count has partitions shared by several CTAs of
    the head kernel and CTAs that carry their sums across tiles."""
    w = replace(ngc_inputs.shrink(ngc_inputs.WORKLOADS[name], rows=rows), pattern="sets")
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    l = w.n_params
    t = ngc_inputs.set_times(w.n, w.levels[-1] + 1, [0, 2, 5])
    outs = []
    for _ in range(3):
        coded = torch.empty((w.n, l), dtype=coded_torch_dtype(p.coded_dtype(m)), device="cuda")
        grad = torch.empty(l, dtype=torch.float32, device="cuda")
        p.step(m, theta, X, y, t, coded, grad)
        torch.cuda.synchronize()
        outs.append((coded.cpu(), grad.cpu()))
    for c, g in outs[1:]:
        assert torch.equal(c, outs[0][0]) and torch.equal(g, outs[0][1])


@pytest.mark.parametrize("name,rows,tol", [("lsq100", 64, 1e-5), ("mlp30", 200, 1e-2)])
def test_step_from_host_buffers_matches_the_device_step(name, rows, tol):
    """ngc_step_host (host buffers in, host gradient out: the end-to-end entry point the benchmark times) gives the
    bits of ngc_step on device copies of the same buffers, also while another data matrix is prepared on the plan."""
    from dataclasses import replace
    w = replace(ngc_inputs.shrink(ngc_inputs.WORKLOADS[name], rows=rows), pattern="sets")
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    l = w.n_params
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    cdt = torch.float64 if p.coded_dtype(m) == ngc.NGC_F64 else torch.float32
    coded = torch.empty((w.n, l), dtype=cdt, device="cuda")
    grad = torch.empty(l, dtype=torch.float32, device="cuda")
    p.prepare_data(m, X)                                    # the host path must not pick this copy up for other data
    Xh = (X.float() * 0.5).to(X.dtype).cpu().pin_memory()   # other contents than the prepared matrix
    yh, thh = y.cpu().pin_memory(), theta.cpu().pin_memory()
    gh = torch.empty(l, dtype=torch.float32).pin_memory()
    for stragglers in ([], [2], list(range(w.levels[-1]))):
        t = ngc_inputs.set_times(w.n, w.levels[-1] + 1, stragglers)
        info_h = p.step_host(m, thh, Xh, yh, t, gh)
        info_d = p.step(m, theta, Xh.cuda(), y, t, coded, grad)
        torch.cuda.synchronize()
        assert info_h.layer == info_d.layer and list(info_h.responsive()) == list(info_d.responsive())
        assert torch.equal(gh, grad.cpu())
        G = oracle_G(w, Xh.cuda(), y, theta)
        assert rel_l2(gh.numpy(), G.sum(axis=0)) < tol
    assert p.device_status() < 1e-6
