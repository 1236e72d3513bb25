"""The sharded entry points on one GPU: the shards of one problem are run one after the other in this process,
the halo rows are copied where `ShardLayout.halo` says the exchange would put them, and the shares of the decode
are added in fp64 as the all-reduce would.  Checked against the CPU oracle and against the unsharded ngc_step.
(No process waits on another one here; the exchange itself is tested with gloo ranks on CPU.)"""
import numpy as np
import pytest
import torch

import ngc_inputs
import paper_2212_08580_b200 as ngc
from oracle import ngc_oracle as orc
from paper_2212_08580_b200.sharded import ShardLayout, ShardedStep
from tests._util import coded_torch_dtype, model_of, oracle_G, rel_l2

pytestmark = pytest.mark.gpu


def _case(kind, x_dtype, n, levels, rows, d, index, C=0, hidden=0):
    return ngc_inputs.Workload(f"shard{index}", 900 + index, n, tuple(levels), kind, rows, d, x_dtype,
                               n_classes=C, hidden=hidden, pattern="sets")


CASES = [
    (_case("lsq", "bf16", 10, [1, 2, 5], 96, 2048, 0), 3, 1e-5),
    (_case("logistic", "f32", 7, [1, 3], 130, 512, 1), 2, 1e-5),
    (_case("softmax", "bf16", 6, [1, 2], 256, 128, 2, C=256), 2, 1e-2),
    (_case("mlp", "f32", 5, [0, 2], 200, 64, 3, C=10, hidden=128), 4, 1e-2),
]


@pytest.mark.parametrize("w,world,tol", CASES)
def test_shards_run_in_turn_reproduce_the_unsharded_step(w, world, tol):
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    l = w.n_params
    lay = ShardLayout(w.n, world)
    pl = orc.plan(w.n, list(w.levels), w.seed)
    G = oracle_G(w, X, y, theta)
    g_full = G.sum(axis=0)
    ref = ngc.Plan(w.n, w.levels, seed=w.seed)
    cdt = coded_torch_dtype(ref.coded_dtype(m))
    coded_ref = torch.empty((w.n, l), dtype=cdt, device="cuda")
    grad_ref = torch.empty(l, dtype=torch.float32, device="cuda")
    shards = [ShardedStep(ngc, w, X[lay.first(r): lay.first(r) + lay.count(r)].contiguous(),
                          y[lay.first(r): lay.first(r) + lay.count(r)].contiguous(), r, world, "cuda")
              for r in range(world)]
    rng = np.random.default_rng(w.seed)
    # single partitions / coded rows of the MLP against the pure fp64 oracle carry the ReLU decisions that flip
    # under bf16 operands (bounded as in test_gpu_mlp.py); what proves the sharding is the bit-equality with the
    # unsharded encode below
    tol_rows = 5e-2 if w.kind == "mlp" else tol
    for layer, s in enumerate(w.levels):
        stragglers = sorted(int(v) for v in rng.choice(w.n, size=s, replace=False))
        t = ngc_inputs.set_times(w.n, w.levels[-1] + 1, stragglers)
        info = ref.step(m, theta, X, y, t, coded_ref, grad_ref)
        assert info.sigma == s
        S = info.responsive()
        for st in shards:                                     # 1. own partial gradients
            st.plan.shard_gradients(m, theta, st.X, st.y, st.n_local, st.G, st.ld)
        torch.cuda.synchronize()
        for st in shards:                                     # partial gradients against the oracle's
            got = st.G[: st.n_local, :l].cpu().numpy()
            for r in range(st.n_local):
                assert rel_l2(got[r], G[st.first + r]) < tol_rows
        for st in shards:                                     # 2. the halo, copied where the exchange would put it
            for src, lrow, take, hrow in lay.halo(st.rank, s):
                st.G[st.n_local + hrow: st.n_local + hrow + take].copy_(shards[src].G[lrow: lrow + take])
        total = torch.zeros(l, dtype=torch.float64, device="cuda")
        want_coded = orc.encode(pl["B"][layer], G)
        for st in shards:                                     # 3. encode + share of the decode
            st.plan.shard_encode_decode(m, layer, st.first, st.n_local, st.G, st.ld, S, st.coded, st.partial)
            torch.cuda.synchronize()
            got = st.coded[: st.n_local].cpu().numpy()
            for r in range(st.n_local):
                assert rel_l2(got[r], want_coded[st.first + r]) < tol_rows, (layer, st.rank, r)
                # the same bits as the unsharded encode wherever the summation order is the same (one slot per group)
                if w.kind in ("softmax", "mlp"):
                    assert torch.equal(st.coded[r], coded_ref[st.first + r])
            total += st.partial.double()                      # 4. what the all-reduce adds up
            assert st.plan.device_status() < 1e-6
        grad = total.float()
        assert rel_l2(grad.cpu().numpy(), g_full) < tol
        assert rel_l2(grad.cpu().numpy(), grad_ref.cpu().numpy()) < (1e-6 if tol < 1e-3 else 1e-5)


def test_single_rank_sharded_step_is_the_whole_problem():
    w = _case("lsq", "bf16", 6, [1, 2], 64, 1024, 9)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    st = ShardedStep(ngc, w, X, y, 0, 1, "cuda")
    G = oracle_G(w, X, y, theta)
    for stragglers in ([], [4], [0, 5]):
        info = st.step(theta, ngc_inputs.set_times(w.n, 3, stragglers))
        torch.cuda.synchronize()
        assert info.sigma == (1 if len(stragglers) < 2 else 2)
        assert rel_l2(st.grad.cpu().numpy(), G.sum(axis=0)) < 1e-5


def test_one_plan_serving_different_shards_in_turn_reloads_its_code_rows():
    """The rows of B a shard needs stay on the device per level; a plan asked for another shard must replace them."""
    w = _case("logistic", "f32", 9, [2], 96, 256, 11)
    X, y, theta = ngc_inputs.make_data(w, "cuda")
    m = model_of(w)
    l = w.n_params
    lay = ShardLayout(w.n, 2)
    G = oracle_G(w, X, y, theta)
    p = ngc.Plan(w.n, w.levels, seed=w.seed)
    cdt = coded_torch_dtype(p.coded_dtype(m))
    ld = (l + 3) // 4 * 4
    t = ngc_inputs.set_times(w.n, 3, [1, 7])
    info = p.select(t)
    S, s = info.responsive(), info.sigma
    Gd = torch.zeros((w.n, ld), dtype=torch.float32, device="cuda")
    p.shard_gradients(m, theta, X, y, w.n, Gd, ld)                      # all groups at once: the rows to hand out
    for _ in range(2):                                                  # shard 0, shard 1, shard 0, shard 1
        total = torch.zeros(l, dtype=torch.float64, device="cuda")
        for r in range(2):
            first, cnt = lay.first(r), lay.count(r)
            win = torch.zeros((cnt + s, ld), dtype=torch.float32, device="cuda")
            rows = [(first + i) % w.n for i in range(cnt + s)]
            win.copy_(Gd[rows])
            coded = torch.empty((cnt + s, l), dtype=cdt, device="cuda")
            part = torch.empty(l, dtype=cdt, device="cuda")
            p.shard_encode_decode(m, info.layer, first, cnt, win, ld, S, coded, part)
            torch.cuda.synchronize()
            total += part.double()
        assert rel_l2(total.cpu().numpy(), G.sum(axis=0)) < 1e-5
