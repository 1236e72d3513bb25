"""GPU parity of the MLP path (tcgen05 contractions + fused back-propagation epilogue) against the CPU oracle."""
import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import coded_torch_dtype, group_G, model_of, oracle_G, rel_l2

pytestmark = pytest.mark.gpu

TOL = 1e-2          # relative L2, bf16 tensor-core operands


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
        got = coded.cpu().numpy()
        assert np.isfinite(got).all()
        for i in range(n):
            # every block of the flattened gradient on its own scale: dW1, db1, dW2, db2
            for a, b in ((0, o1), (o1, o2), (o2, o3), (o3, l)):
                assert rel_l2(got[i, a:b], want[i, a:b]) < TOL, (layer, i, a, rel_l2(got[i, a:b], want[i, a:b]))
        for trial in range(2):
            stragglers = rng.choice(n, size=s, replace=False) if trial else np.arange(s)
            S = np.array(sorted(set(range(n)) - set(int(v) for v in stragglers)), dtype=np.int32)
            p.decode(layer, S, coded, cdt, l, grad)
            torch.cuda.synchronize()
            assert rel_l2(grad.cpu().numpy(), g_full) < TOL
