"""GPU parity of the softmax-regression path (tcgen05 contractions) against the CPU oracle."""
import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import assert_dense_close, coded_torch_dtype, group_G, model_of, oracle_G, rel_l2

pytestmark = pytest.mark.gpu

TOL = 1e-2          # relative L2, bf16 tensor-core operands


def _workload(n, levels, rows, d, C, index, q=1):
    return ngc_inputs.Workload(f"softmax_case{index}", 500 + index, n * q, tuple(levels), "softmax", rows, d, "bf16",
                               n_classes=C, pattern="sets")


CASES = [
    # n, levels, rows, d, C, partitions per worker
    (3, [0], 128, 64, 64, 1),          # one row block, one K chunk: coded == G
    (3, [0], 256, 256, 256, 1),        # full-width classes, several K chunks and stages
    (5, [0, 2], 300, 192, 80, 1),      # ragged rows (300 = 2*128+44), ragged feature block, C not a multiple of 64
    (6, [1, 3], 1000, 512, 128, 1),
    (4, [1], 130, 128, 16, 2),         # k = 2 n, smallest class count
    (4, [1], 520, 1032, 256, 1),       # CTA-pair kernels: ragged 256-row blocks, five feature blocks (the last 8 wide)
    (2, [1], 200, 128, 256, 2),        # k = 2 n with full-width classes, less than one 256-row block
    (2, [0], 256, 64, 256, 2),         # ... exactly one block, a single K chunk in the forward pass
    (90, [1], 192, 1032, 256, 1),      # backward units on the CTA pairs in four and five rounds: whole passes, halves
                                       # and ragged passes after one another, the one-accumulator units taking turns
]


@pytest.mark.parametrize("n,levels,rows,d,C,q", CASES)
def test_softmax_grad_encode_decode_match_oracle(n, levels, rows, d, C, q):
    w = _workload(n, levels, rows, d, C, rows % 97 + C, q)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    p = ngc.Plan(n, levels, n_partitions=n * q, seed=w.seed)
    pl = orc.plan(n, levels, w.seed)
    G = group_G(oracle_G(w, X, y, theta), q)
    g_full = G.sum(axis=0)
    l = d * C
    cdt = p.coded_dtype(m)
    coded = torch.empty((n, l), dtype=coded_torch_dtype(cdt), device="cuda")
    grad = torch.empty(l, dtype=torch.float32, device="cuda")
    rng = np.random.default_rng(w.seed)
    for layer, s in enumerate(levels):
        coded.fill_(float("nan"))
        p.grad_encode(m, theta, X, y, layer, coded)
        torch.cuda.synchronize()
        assert p.device_status() < 1e-6
        want = orc.encode(pl["B"][layer], G)
        got = coded.cpu().numpy()
        for i in range(n):
            # the whole row, every 128-feature x 256-class block of it, and the largest single error
            assert_dense_close(got[i], want[i], C, TOL, (layer, i))
        for trial in range(2):
            stragglers = rng.choice(n, size=s, replace=False) if trial else np.arange(s)
            S = np.array(sorted(set(range(n)) - set(int(v) for v in stragglers)), dtype=np.int32)
            p.decode(layer, S, coded, cdt, l, grad)
            torch.cuda.synchronize()
            assert_dense_close(grad.cpu().numpy(), g_full, C, TOL, (layer, "decoded"))
