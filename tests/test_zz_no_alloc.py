"""ngc_grad_encode_static against ngc_grad_encode, through the C ABI.

The static variant exists for programs that may not allocate device memory when they call the
library (their own pool owns the whole GPU, or an allocation's device-wide stall is unaffordable).
It must give the same coded gradients as the allocating entry point, call after call, although all
calls share one fixed scratch array that still holds the previous call's data.
Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.
"""
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from tests._util import coded_torch_dtype, model_of, oracle_G, rel_l2

pytestmark = pytest.mark.gpu

TOL = 1e-5   # relative L2, the tolerance of the other fp32-path tests


def _case(kind, x_dtype, n, levels, rows, d, index):
    return ngc_inputs.Workload(f"static{index}", 300 + index, n, tuple(levels), kind, rows, d, x_dtype)


def test_static_variant_matches_allocating_entry_point_twice_in_a_row():
    cases = [_case("logistic", "f32", 20, [1, 2, 4], 333, 4096, 0),    # first call on this device
             _case("lsq", "bf16", 6, [2, 3], 150, 8192, 1)]            # second call: other shape, stale scratch
    for w in cases:
        X, y, theta = ngc_inputs.make_data(w, "cuda")
        m = model_of(w)
        ref_plan = ngc.Plan(w.n, w.levels, seed=w.seed)
        static_plan = ngc.Plan(w.n, w.levels, seed=w.seed)             # never allocates on the device
        cdt = ref_plan.coded_dtype(m)
        status = torch.full((1,), 7, dtype=torch.int32, device="cuda")
        G = oracle_G(w, X, y, theta)                                   # the CPU oracle, from the same bits
        B = orc.plan(w.n, list(w.levels), w.seed)["B"]
        for layer in range(len(w.levels)):
            want = torch.empty((w.n, w.d), dtype=coded_torch_dtype(cdt), device="cuda")
            got = torch.full_like(want, float("nan"))
            ref_plan.grad_encode(m, theta, X, y, layer, want)
            static_plan.grad_encode_static(m, theta, X, y, layer, got, status)   # (first call: loads the module)
            torch.cuda.synchronize()
            # nothing is allocated or freed on the device: the driver's free-memory figure does not move across
            # further calls (torch's caching allocator is left alone in between)
            free0, _ = torch.cuda.mem_get_info()
            static_plan.grad_encode_static(m, theta, X, y, layer, got, status)
            torch.cuda.synchronize()
            free1, _ = torch.cuda.mem_get_info()
            assert free1 == free0
            assert int(status.item()) == 0
            assert static_plan.workspace_bytes() == 0
            want_oracle = orc.encode(B[layer], G)
            for i in range(w.n):
                assert rel_l2(got[i].cpu().numpy(), want[i].cpu().numpy()) < TOL
                assert rel_l2(got[i].cpu().numpy(), want_oracle[i]) < TOL
        # status pointer is optional
        got2 = torch.full_like(got, float("nan"))
        static_plan.grad_encode_static(m, theta, X, y, len(w.levels) - 1, got2)
        torch.cuda.synchronize()
        assert torch.equal(got2, got)


def test_static_variant_refuses_what_does_not_fit():
    # 128 groups x 2 slots x 16384 floats = 16 MiB of partial gradients > the 8 MiB array
    w = _case("lsq", "bf16", 128, [1], 4, 16384, 2)
    X = torch.zeros((w.n, w.rows, w.d), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((w.n, w.rows), device="cuda")
    theta = torch.zeros(w.d, device="cuda")
    coded = torch.zeros((w.n, w.d), dtype=torch.float64, device="cuda")
    p = ngc.Plan(w.n, w.levels, seed=1)
    with pytest.raises(ngc.NgcError) as e:
        p.grad_encode_static(model_of(w), theta, X, y, 0, coded)
    assert e.value.status == -7
    # softmax / MLP are not offered by this entry point
    with pytest.raises(ngc.NgcError):
        p.grad_encode_static(ngc.Model.make("softmax", "bf16", 4, 16384, 8), theta, X, y, 0, coded)
