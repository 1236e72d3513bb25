"""GPU parity of the least-squares / logistic path against the CPU oracle, through the C ABI."""
import itertools

import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import coded_torch_dtype, group_G, model_of, oracle_G, rel_l2, to_np64

pytestmark = pytest.mark.gpu

TOL = 1e-5          # relative L2, fp32 paths


def _workload(kind, x_dtype, n, levels, rows, d, index):
    return ngc_inputs.Workload(f"case{index}", 100 + index, n, tuple(levels), kind, rows, d, x_dtype)


CASES = [
    # kind, dtype, n, levels, rows, d, partitions-per-worker
    ("lsq", "f32", 6, [1, 2, 3], 777, 1000, 1),          # ragged rows and ragged vectors (1 vector / thread)
    ("logistic", "f32", 20, [1, 2, 4], 301, 4096, 1),    # 2 vectors / thread, 4-row tiles
    ("lsq", "f32", 5, [0, 2], 130, 8192, 1),             # 4 vectors / thread, tolerance 0 listed
    ("lsq", "bf16", 10, [1, 2, 5], 203, 16384, 1),       # the wide bf16 shape
    ("logistic", "bf16", 7, [1, 3], 517, 2056, 1),       # ragged bf16
    ("lsq", "bf16", 8, [2], 64, 8192, 1),                # single component code (plain gradient code)
    ("lsq", "f32", 4, [1, 2], 50, 256, 3),               # k = 3 n: atomic task = 3 partitions
    ("logistic", "f32", 3, [1], 1, 4, 1),                # one row, one vector
    ("lsq", "f32", 128, [1, 32], 3, 64, 1),              # the largest n and the largest tolerance the library takes
    ("lsq", "bf16", 2, [0, 1], 5000, 16384, 1),          # many rows per CTA range, widest rows
    ("logistic", "bf16", 6, [1, 2], 75, 16384, 1),       # two-row tiles (one barrier per tile) with the sigmoid, odd row count
    ("logistic", "f32", 5, [1], 33, 8192, 1),            # the same path on fp32 rows
]


@pytest.mark.parametrize("kind,x_dtype,n,levels,rows,d,q", CASES)
def test_grad_encode_and_decode_match_oracle(kind, x_dtype, n, levels, rows, d, q):
    w = _workload(kind, x_dtype, n * q, levels, rows, d, len(levels) * 7 + d % 97)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(n, levels, n_partitions=n * q, seed=w.seed)
    pl = orc.plan(n, levels, w.seed)
    G = group_G(oracle_G(w, X, y, theta), q)
    g_full = G.sum(axis=0)
    cdt = p.coded_dtype(m)
    coded = torch.empty((n, d), dtype=coded_torch_dtype(cdt), device="cuda")
    grad = torch.empty(d, dtype=torch.float32, device="cuda")
    rng = np.random.default_rng(w.seed)
    for l, s in enumerate(levels):
        coded.fill_(float("nan"))
        p.grad_encode(m, theta, X, y, l, coded)
        torch.cuda.synchronize()
        want = orc.encode(pl["B"][l], G)
        got = coded.cpu().numpy()
        for i in range(n):
            assert rel_l2(got[i], want[i]) < TOL, (l, i)
        for trial in range(3):
            stragglers = rng.choice(n, size=s, replace=False) if trial else np.arange(s)
            S = np.array(sorted(set(range(n)) - set(int(v) for v in stragglers)), dtype=np.int32)
            grad.fill_(float("nan"))
            p.decode(l, S, coded, cdt, d, grad)
            torch.cuda.synchronize()
            a = orc.decode_vector(pl["B"][l], S)
            assert rel_l2(grad.cpu().numpy(), orc.decode(a, want)) < TOL
            assert rel_l2(grad.cpu().numpy(), g_full) < TOL          # the main pin: the uncoded full gradient
    assert p.device_status() < 1e-8
    assert p.launch_count() > 0


def test_tiny_brute_force_all_straggler_sets():
    w = ngc_inputs.WORKLOADS["tiny"]
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    pl = orc.plan(w.n, list(w.levels), w.seed)
    Xn, yn, thn = to_np64(X), to_np64(y), to_np64(theta)
    g_full = orc.full_gradient("lsq", Xn, yn, thn)
    coded = torch.empty((w.n, w.d), dtype=torch.float64, device="cuda")
    grad = torch.empty(w.d, dtype=torch.float32, device="cuda")
    n_tasks = w.levels[-1] + 1
    for size in range(0, 3):
        for stragglers in itertools.combinations(range(w.n), size):
            t = ngc_inputs.set_times(w.n, n_tasks, stragglers)
            info = p.step(m, theta, X, y, t, coded, grad)
            torch.cuda.synchronize()
            want = orc.step(pl, "lsq", Xn, yn, thn, t, 0.0, 0.0)
            assert info.layer == want["level"] and np.array_equal(info.responsive(), want["S"])
            assert info.latency == want["latency"]
            assert np.array_equal(np.array(info.tasks_done[: w.n]), want["tasks_done"])
            assert rel_l2(coded.cpu().numpy(), want["coded"]) < TOL
            assert rel_l2(grad.cpu().numpy(), want["grad"]) < TOL
            assert rel_l2(grad.cpu().numpy(), g_full) < TOL
    with pytest.raises(ngc.NgcError) as e:
        p.step(m, theta, X, y, ngc_inputs.set_times(w.n, n_tasks, [0, 1, 2]), coded, grad)
    assert e.value.status == -2


@pytest.mark.parametrize("n,levels,seed", [(20, [1, 2, 4], 1), (50, [1, 3, 5, 10], 2), (100, [1, 2, 5, 10], 3),
                                           (30, [1, 2, 3, 6], 4), (128, [32], 5), (9, [0], 6)])
def test_decode_vectors_batched(n, levels, seed):
    p = ngc.Plan(n, levels, seed=221208580 + seed)
    pl = orc.plan(n, levels, 221208580 + seed)
    rng = np.random.default_rng(seed)
    for l, s in enumerate(levels):
        batch = 9
        S = np.stack([np.array(sorted(set(range(n)) - set(rng.choice(n, size=s, replace=False).tolist())),
                               dtype=np.int32) for _ in range(batch)])
        S[0] = np.arange(s, n)                      # contiguous stragglers 0..s-1
        a, res = p.decode_vectors(l, S)
        B = pl["B"][l]
        for b in range(batch):
            want = orc.decode_vector(B, S[b])
            assert set(np.nonzero(a[b])[0]) <= set(S[b].tolist())
            scale = max(1.0, np.abs(want).sum())
            assert np.max(np.abs(a[b] @ B - 1.0)) < 1e-9 * scale     # Definition 1: a B = 1
            assert abs(res[b] - np.max(np.abs(a[b] @ B - 1.0))) < 1e-10 * scale
            assert rel_l2(a[b], want) < 1e-7                           # unique solution, two different algorithms
        one = p.decode_vector(l, S[1])
        assert np.array_equal(one, a[1])


def test_decode_uses_smallest_indices_when_more_respond():
    n, levels = 8, [2]
    p = ngc.Plan(n, levels, seed=3)
    a_all = p.decode_vector(0, np.arange(n, dtype=np.int32))
    a_first = p.decode_vector(0, np.arange(n - 2, dtype=np.int32))
    assert np.array_equal(a_all, a_first) and a_all[-1] == 0 and a_all[-2] == 0


def test_device_argument_errors():
    p = ngc.Plan(4, [1, 2], seed=1)
    m = ngc.Model.make("lsq", "f32", 8, 32)
    X = torch.zeros((4, 8, 32), device="cuda")
    y = torch.zeros((4, 8), device="cuda")
    th = torch.zeros(32, device="cuda")
    coded = torch.zeros((4, 32), dtype=torch.float64, device="cuda")
    grad = torch.zeros(32, device="cuda")
    with pytest.raises(ngc.NgcError):
        p.grad_encode(m, th, X, y, 2, coded)                       # layer out of range
    with pytest.raises(ngc.NgcError):
        p.grad_encode(ngc.Model.make("lsq", "f32", 8, 30), th, X, y, 0, coded)   # rows not whole 16-byte vectors
    with pytest.raises(ngc.NgcError):
        p.decode(0, np.array([0, 1], dtype=np.int32), coded, ngc.NGC_F64, 32, grad)   # too few responders
    with pytest.raises(ngc.NgcError):
        p.decode(0, np.array([0, 2, 1], dtype=np.int32), coded, ngc.NGC_F64, 32, grad)  # not sorted
    with pytest.raises(ngc.NgcError):
        p.decode(0, np.array([0, 1, 4], dtype=np.int32), coded, ngc.NGC_F64, 32, grad)  # out of range
    # the context is still usable afterwards
    p.grad_encode(m, th, X, y, 0, coded)
    torch.cuda.synchronize()
    assert float(coded.abs().max()) == 0.0


def test_runs_are_bitwise_reproducible():
    w = _workload("logistic", "f32", 12, [1, 3], 400, 2048, 77)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    outs = []
    for _ in range(3):
        coded = torch.empty((w.n, w.d), dtype=torch.float64, device="cuda")
        p.grad_encode(m, theta, X, y, 1, coded)
        torch.cuda.synchronize()
        outs.append(coded.cpu())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
