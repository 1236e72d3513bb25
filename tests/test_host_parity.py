"""Host-side logic of the library against the CPU oracle (no GPU needed): the code matrices, the
task schedule and the stopping rule must agree BIT FOR BIT; plus the C-ABI surface itself."""
import ctypes
import os
import re

import numpy as np
import pytest

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "ngc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(ngc_[a-z_0-9]+)\s*\(", text))
    assert {"ngc_plan", "ngc_grad_encode", "ngc_decode", "ngc_step"} <= names
    lib = ctypes.CDLL(ngc.lib_path())
    for name in sorted(names):
        assert hasattr(lib, name), name


@pytest.mark.parametrize("name", list(ngc_inputs.WORKLOADS))
def test_B_and_schedule_bit_exact(name):
    w = ngc_inputs.WORKLOADS[name]
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    pl = orc.plan(w.n, list(w.levels), w.seed)
    for l in range(len(w.levels)):
        assert np.array_equal(p.B_dense(l), pl["B"][l])
    order, tpl = p.schedule()
    assert np.array_equal(order, pl["schedule"]) and order.dtype == np.int32
    assert np.array_equal(tpl, pl["tasks_per_level"])


@pytest.mark.parametrize("n,levels,seed", [(1, [0], 5), (2, [0, 1], 6), (8, [0, 1, 2, 3], 7), (13, [2, 5, 12], 8),
                                           (128, [1, 32], 9), (37, [0, 7, 19], 2 ** 63 + 11)])
def test_B_bit_exact_odd_shapes(n, levels, seed):
    p = ngc.Plan(n, levels, seed=seed)
    pl = orc.plan(n, levels, seed)
    for l in range(len(levels)):
        assert np.array_equal(p.B_dense(l), pl["B"][l])


@pytest.mark.parametrize("name", list(ngc_inputs.WORKLOADS))
def test_selection_bit_exact(name):
    w = ngc_inputs.WORKLOADS[name]
    p = ngc.Plan(w.n, w.levels, seed=w.seed, gamma=0.75, eps=0.1)
    undecodable = 0
    for it in range(200):
        t = ngc_inputs.pattern_times(w, it)
        want = orc.select(t, list(w.levels), 0.75, 0.1)
        if want is None:
            with pytest.raises(ngc.NgcError) as e:
                p.select(t)
            assert e.value.status == -2
            undecodable += 1
            continue
        got = p.select(t)
        assert got.layer == want["level"] and got.sigma == want["sigma"] and got.nS == len(want["S"])
        assert np.array_equal(got.responsive(), want["S"])
        assert got.latency == want["latency"]                       # same fp64 bits
        assert np.array_equal(np.array(got.tasks_done[: w.n]), want["tasks_done"])
    if w.p_fail == 0 and w.pattern == "times":
        assert undecodable == 0


def test_selection_ties_and_dead_workers():
    p = ngc.Plan(6, [0, 1, 3], seed=1)
    rng = np.random.default_rng(0)
    for _ in range(300):
        t = rng.integers(1, 3, size=(6, 4)).astype(np.float64)      # many exact ties
        t[rng.random(6) < 0.25, :] = np.inf
        want = orc.select(t, [0, 1, 3], 0.0, 0.0)
        if want is None:
            with pytest.raises(ngc.NgcError):
                p.select(t)
            continue
        got = p.select(t)
        assert (got.layer, list(got.responsive()), got.latency) == (want["level"], list(want["S"]), want["latency"])
        assert np.array_equal(np.array(got.tasks_done[:6]), want["tasks_done"])


def test_argument_errors():
    with pytest.raises(ngc.NgcError):
        ngc.Plan(4, [2, 1])                    # not increasing
    with pytest.raises(ngc.NgcError):
        ngc.Plan(4, [4])                       # s must be < n
    with pytest.raises(ngc.NgcError):
        ngc.Plan(4, [1], n_partitions=6)       # k not a multiple of n
    with pytest.raises(ngc.NgcError):
        ngc.Plan(129, [1])                     # n above NGC_MAX_N
    p = ngc.Plan(4, [1, 2])
    bad = np.ones((4, 3)); bad[0, 0] = -1.0
    with pytest.raises(ngc.NgcError):
        p.select(bad)
    bad[0, 0] = np.nan
    with pytest.raises(ngc.NgcError):
        p.select(bad)
    assert p.num_params(ngc.Model.make("mlp", "f32", 10, 784, 10, 512)) == 407050
    assert p.num_params(ngc.Model.make("softmax", "bf16", 10, 1024, 256)) == 262144
    assert p.coded_dtype(ngc.Model.make("lsq", "f32", 10, 32)) == ngc.NGC_F64
    assert p.coded_dtype(ngc.Model.make("mlp", "f32", 10, 784, 10, 512)) == ngc.NGC_F32
    p.set_coded_dtype(ngc.NGC_F32)
    assert p.coded_dtype(ngc.Model.make("lsq", "f32", 10, 32)) == ngc.NGC_F32
    # Monte Carlo of the stopping rule: one of the two outputs may be left out, not both (checked before any launch)
    lib = ngc.load_library()
    assert lib.ngc_latency_mc(p._h, 1, 16, 0.5, 0.5, 0.05, None, None, None) == -1
    assert lib.ngc_latency_mc(p._h, 1, 0, 0.5, 0.5, 0.05, None, None, None) == -1
    assert lib.ngc_selftest_wait_timeout(p._h, 0, None) == -1
    assert lib.ngc_selftest_wait_timeout(None, 1000, None) == -1


def test_sample_times_model():
    # Section II-D: shift + Exp(rate) per task, workers fail independently
    t = ngc.sample_times(42, 100, 11, 1.0, 2.0, 0.05)
    dead = np.isinf(t).all(axis=1)
    assert np.array_equal(np.isinf(t).any(axis=1), dead)
    alive = t[~dead]
    assert alive.min() >= 1.0 and abs(alive.mean() - 1.5) < 0.05
    big = ngc.sample_times(43, 128, 33, 0.0, 1.0, 0.05)
    assert 0.01 < np.isinf(big).all(axis=1).mean() < 0.12
    assert np.array_equal(t, ngc.sample_times(42, 100, 11, 1.0, 2.0, 0.05))
