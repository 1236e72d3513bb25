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
