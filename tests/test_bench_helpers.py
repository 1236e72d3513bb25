"""Host-side arithmetic of the benchmark (no GPU): the algorithmic work per launch that the roofline fractions divide
by, the clock sampler's bookkeeping and the reduced-copy CPU leg."""
import numpy as np
import torch

import bench
import ngc_inputs


def test_algorithmic_work_per_launch():
    W = ngc_inputs.WORKLOADS
    # data matrix and labels once, theta, the coded matrix (fp64 for the GEMV workloads)
    assert bench.algorithmic_bytes(W["logistic20"], 8) == 20 * 8192 * (4096 * 4 + 4) + 4 * 4096 + 20 * 4096 * 8 == 2_685_681_664
    assert bench.algorithmic_bytes(W["lsq100"], 8) == 100 * 2000 * (16384 * 2 + 4) + 4 * 16384 + 100 * 16384 * 8 == 6_567_572_736
    # two contractions of 2 flops per multiply-add each
    assert bench.algorithmic_flops(W["softmax50"]) == 4 * 50 * 4096 * 1024 * 256 == 214_748_364_800
    assert bench.algorithmic_flops(W["mlp30"]) == 60000 * (4 * 784 * 512 + 6 * 512 * 10) == 98_181_120_000


def test_roofline_object_uses_the_measured_peaks():
    W = ngc_inputs.WORKLOADS
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops_sustained": 1400.0}
    r = bench.roofline_of(W["lsq100"], True, 10.0, 10, peaks, "measured", 123)
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["traffic"] == 123
    assert abs(r["achieved"] - 6_567_572_736 / 1e-3 / 1e9) < 1e-6 and abs(r["frac"] - r["achieved"] / 6500.0) < 1e-12
    r = bench.roofline_of(W["softmax50"], False, 2.0, 10, peaks, "measured", None)
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and r["peak"] == 1400.0
    assert abs(r["achieved"] - 214_748_364_800 / 0.2e-3 / 1e12) < 1e-6


def test_cpu_leg_on_a_reduced_copy_decodes_the_reduced_problem():
    # the reference arm's step: every partition cut to its first rows, a full oracle step on that copy
    w = ngc_inputs.WORKLOADS["tiny"]
    X, y, theta = ngc_inputs.make_data(w, "cpu")
    t = ngc_inputs.set_times(w.n, w.levels[-1] + 1, [1])
    secs, spent, g = bench.oracle_reduced_step(w, X, y, theta, t, 16)
    from oracle import ngc_oracle as orc
    want = orc.full_gradient("lsq", X[:, :16].double().numpy(), y[:, :16].double().numpy(), theta.double().numpy())
    assert np.linalg.norm(g - want) <= 1e-9 * np.linalg.norm(want)
    assert secs >= spent > 0.0                         # the gradient part is scaled up by rows / rows_r = 4
    assert 1 <= bench.rows_within_budget(w, X[:, :8], y[:, :8], theta, t, 1e-9) <= w.rows
    assert bench.rows_within_budget(w, X[:, :8], y[:, :8], theta, t, 1e9) == w.rows


def test_replicas_differ_only_in_their_seed():
    w = ngc_inputs.WORKLOADS["tiny"]
    r1 = bench.replica_workload(w, 1)
    assert (r1.n, r1.levels, r1.rows, r1.d) == (w.n, w.levels, w.rows, w.d) and r1.seed != w.seed
    assert not torch.equal(ngc_inputs.make_data(w)[0], ngc_inputs.make_data(r1)[0])
