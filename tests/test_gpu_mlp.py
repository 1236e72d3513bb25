"""GPU parity of the MLP path (tcgen05 contractions + fused back-propagation epilogue) against the CPU oracle."""
import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import assert_dense_close, coded_torch_dtype, group_G, model_of, oracle_G, rel_l2

pytestmark = pytest.mark.gpu

TOL = 1e-2          # relative L2, bf16 tensor-core operands
TOL_PURE_ROW = 5e-2  # one worker's coded dW1 against the oracle that decides the ReLU derivative in fp64: the units
                     # whose pre-activation changes sign under bf16 operands (about 7e-4 of them) each move one
                     # entry of delta1 by O(1); measured about 2e-2 on a single partition


def _workload(n, levels, rows, d, hidden, C, index, q=1):
    return ngc_inputs.Workload(f"mlp_case{index}", 700 + index, n * q, tuple(levels), "mlp", rows, d, "f32",
                               n_classes=C, hidden=hidden, pattern="sets")


CASES = [
    # n, levels, rows, d, hidden, C, partitions per worker
    (3, [0], 128, 64, 64, 10, 1),        # one tile, one accumulator: coded == G
    (3, [0], 256, 784, 512, 10, 1),      # the 784-512-10 shape: two accumulators, ragged K (785 -> 13 chunks)
    (5, [0, 2], 300, 200, 256, 7, 1),    # ragged rows, odd class count
    (4, [1], 130, 128, 32, 3, 2),        # k = 2 n, narrow hidden layer
    (3, [1], 77, 72, 512, 16, 1),        # widest class count
    (10, [1], 2000, 64, 128, 10, 1),     # 160 head tiles on 148 CTAs: output-layer sums carried across tiles and CTAs
    (3, [0], 200, 64, 192, 5, 1),        # hidden not a multiple of 128: output-layer gradient by its own contraction
]


@pytest.mark.parametrize("n,levels,rows,d,hidden,C,q", CASES)
def test_mlp_grad_encode_decode_match_oracle(n, levels, rows, d, hidden, C, q):
    w = _workload(n, levels, rows, d, hidden, C, rows % 89 + hidden % 7 + C, q)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    g = torch.Generator(device="cuda").manual_seed(w.seed)
    theta = theta + 0.05 * torch.randn(theta.shape, generator=g, device="cuda")      # non-zero biases
    m = model_of(w)
    p = ngc.Plan(n, levels, n_partitions=n * q, seed=w.seed)
    pl = orc.plan(n, levels, w.seed)
    G = group_G(oracle_G(w, X, y, theta), q)          # the plain fp64 definition
    g_full = G.sum(axis=0)
    # Coded rows are compared with the ReLU derivative decided in the kernel's precision (bf16 operands):
    # a unit whose pre-activation changes sign under bf16 rounding moves one entry of delta1 by O(1).
    th = theta.double().cpu()
    W1 = th[: d * hidden].view(d, hidden).bfloat16().double()
    b1 = th[d * hidden: d * hidden + hidden].bfloat16().double()
    Gm = []
    for j in range(n * q):
        mask = (X[j].cpu().bfloat16().double() @ W1 + b1 > 0).numpy()
        Gm.append(orc.grad_mlp(X[j].double().cpu().numpy(), y[j].cpu().numpy(), th.numpy(), hidden, C, relu_mask=mask))
    Gm = group_G(np.stack(Gm), q)
    gm_full = Gm.sum(axis=0)
    l = w.n_params
    cdt = p.coded_dtype(m)
    coded = torch.empty((n, l), dtype=coded_torch_dtype(cdt), device="cuda")
    grad = torch.empty(l, dtype=torch.float32, device="cuda")
    rng = np.random.default_rng(w.seed)
    o1, o2, o3 = d * hidden, d * hidden + hidden, d * hidden + hidden + hidden * C
    for layer, s in enumerate(levels):
        coded.fill_(float("nan"))
        p.grad_encode(m, theta, X, y, layer, coded)
        torch.cuda.synchronize()
        assert p.device_status() < 1e-6
        want = orc.encode(pl["B"][layer], Gm)
        want_pure = orc.encode(pl["B"][layer], G)        # ReLU derivative decided in fp64
        got = coded.cpu().numpy()
        assert np.isfinite(got).all()
        worst_pure = 0.0
        for i in range(n):
            # every block of the flattened gradient on its own scale: dW1, db1, dW2, db2
            for a, b in ((0, o1), (o1, o2), (o2, o3), (o3, l)):
                assert rel_l2(got[i, a:b], want[i, a:b]) < TOL, (layer, i, a, rel_l2(got[i, a:b], want[i, a:b]))
            # dW1 (d x hidden) and dW2 (hidden x C) tile by tile, and their largest single errors
            assert_dense_close(got[i, :o1], want[i, :o1], hidden, TOL, (layer, i, "dW1"))
            assert_dense_close(got[i, o2:o3], want[i, o2:o3], C, TOL, (layer, i, "dW2"))
            # against the unmodified oracle, with its own bound (the parts the mask does not touch at TOL)
            worst_pure = max(worst_pure, rel_l2(got[i, :o2], want_pure[i, :o2]))
            assert rel_l2(got[i, o2:], want_pure[i, o2:]) < TOL
        print(f"mlp coded rows vs pure fp64 oracle, level {layer}: worst [dW1, db1] rel L2 {worst_pure:.2e}")
        assert worst_pure < TOL_PURE_ROW, (layer, worst_pure)
        for trial in range(2):
            stragglers = rng.choice(n, size=s, replace=False) if trial else np.arange(s)
            S = np.array(sorted(set(range(n)) - set(int(v) for v in stragglers)), dtype=np.int32)
            p.decode(layer, S, coded, cdt, l, grad)
            torch.cuda.synchronize()
            gd = grad.cpu().numpy()
            assert rel_l2(gd, g_full) < TOL
            # the whole decoded gradient against the pure fp64 oracle at TOL (above); its first-layer part alone
            # carries the ReLU decisions that flip under bf16 operands (a flipped unit of one sample is an O(1)
            # error in single entries of dW1, which weighs most when partitions have few rows): bounded like the
            # coded rows, and checked tile by tile and entry by entry with the decision matched
            assert rel_l2(gd[:o2], g_full[:o2]) < TOL_PURE_ROW
            assert_dense_close(gd[:o1], gm_full[:o1], hidden, TOL, (layer, "decoded dW1, decision matched"))
            assert_dense_close(gd[o2:o3], g_full[o2:o3], C, TOL, (layer, "decoded dW2"))


def test_data_prepared_once_gives_the_same_bits_and_is_tied_to_its_pointer():
    """ngc_prepare_data: the bf16 copy of the data matrix made once must give exactly what the per-call conversion
    gives, must be used only for the pointer it was made from, and must follow a second call when the data change."""
    w = _workload(6, [1, 2], 300, 784, 512, 10, 41)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    l = w.n_params
    p_ref = ngc.Plan(w.n, w.levels, seed=w.seed)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    want = torch.empty((w.n, l), dtype=torch.float32, device="cuda")
    got = torch.empty_like(want)
    p_ref.grad_encode(m, theta, X, y, 1, want)
    p.prepare_data(m, X)
    assert p.workspace_bytes() >= w.n * w.rows * 792 * 2
    launches0 = p.launch_count()
    p.grad_encode(m, theta, X, y, 1, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    assert p.launch_count() - launches0 == p_ref.launch_count()
    # another tensor with other contents: not the prepared pointer, so converted per call
    X2 = (1.0 - X).contiguous()
    p_ref.grad_encode(m, theta, X2, y, 1, want)
    p.grad_encode(m, theta, X2, y, 1, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    # the contents behind the prepared pointer change: a second call picks them up
    X.copy_(X2)
    p.prepare_data(m, X)
    p.grad_encode(m, theta, X, y, 1, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    # dropped: back to the per-call conversion; other models accept the call and do nothing
    p.prepare_data(m, None)
    p.grad_encode(m, theta, X, y, 1, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    p.prepare_data(ngc.Model.make("lsq", "f32", 8, 64), X)
    assert p.device_status() < 1e-6
