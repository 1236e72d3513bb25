"""N > 1 plumbing of the benchmark on CPU (gloo, world size 2): replicas are independent problems, the
job time is the maximum over ranks, launch counts are summed, and only rank 0 reports."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    import ngc_inputs
    w = bench.replica_workload(ngc_inputs.WORKLOADS["tiny"], rank)
    X, _, _ = ngc_inputs.make_data(w)
    res = {
        "max": bench.rank_max(10.0 + rank, world),
        "sum": bench.rank_sum(4.0, world),
        "seed": w.seed,
        "x0": float(X[0, 0, 0]),
    }
    dist.barrier()
    torch.save(res, os.path.join(out, f"r{rank}.pt"))
    dist.destroy_process_group()


def test_rank_reductions_and_independent_replicas(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = torch.load(tmp_path / "r0.pt")
    r1 = torch.load(tmp_path / "r1.pt")
    assert r0["max"] == r1["max"] == 11.0          # slowest rank decides
    assert r0["sum"] == r1["sum"] == 8.0
    assert r0["seed"] != r1["seed"] and r0["x0"] != r1["x0"]   # each rank its own problem, nothing exchanged


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "2", "--warmup", "1", "--workload", "tiny"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


# ---------------------------------------------------------------- one problem sharded over the ranks
def test_shard_layout_covers_every_window_exactly_once():
    from paper_2212_08580_b200.sharded import ShardLayout
    for n, world in [(4, 2), (7, 2), (7, 3), (20, 8), (100, 8), (5, 5), (6, 1)]:
        lay = ShardLayout(n, world)
        assert sum(lay.count(r) for r in range(world)) == n and lay.first(world) == n
        for g in range(n):
            r = lay.owner(g)
            assert lay.first(r) <= g < lay.first(r) + lay.count(r)
        for s in range(0, min(n, 11)):
            for r in range(world):
                rows = []
                for src, lrow, take, hrow in lay.halo(r, s):
                    assert hrow == len(rows) and 0 <= lrow and lrow + take <= lay.count(src)
                    rows += [lay.first(src) + lrow + t for t in range(take)]
                # the s groups behind the block, in cyclic order
                assert rows == [(lay.first(r) + lay.count(r) + t) % n for t in range(s)]
            # every receive has its matching send
            want = sorted((src, r, lrow, take) for r in range(world) for src, lrow, take, _ in lay.halo(r, s) if src != r)
            have = sorted((r, dst, lrow, take) for r in range(world) for dst, lrow, take in lay.sends(r, s))
            assert want == have


def _shard_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import ngc_oracle as orc
    from paper_2212_08580_b200.sharded import ShardLayout, exchange_halo
    n, levels, rows, d = 7, [1, 3], 6, 5
    rng = np.random.default_rng(5)                       # the same problem on every rank
    X = rng.normal(size=(n, rows, d))
    y = rng.normal(size=(n, rows))
    theta = rng.normal(size=d)
    pl = orc.plan(n, levels, 99)
    g_full = orc.full_gradient("lsq", X, y, theta)
    lay = ShardLayout(n, world)
    lo, cnt = lay.first(rank), lay.count(rank)
    G_own = np.stack([orc.grad_lsq(X[j], y[j], theta) for j in range(lo, lo + cnt)])   # this rank's partitions only
    G_all = orc.partial_gradients("lsq", X, y, theta)
    worst = 0.0
    # rank 0 holds groups 0-2, rank 1 groups 3-6: windows of workers 2 and 6 straddle a boundary; stragglers are
    # taken on either side of it
    cases = [(0, [2]), (0, [3]), (1, [1, 2, 3]), (1, [2, 5, 6]), (1, [0, 3, 4]), (0, [6])]
    for level, stragglers in cases:
        s, B = levels[level], pl["B"][level]
        S = [i for i in range(n) if i not in stragglers]
        Gw = torch.zeros((cnt + s, 8), dtype=torch.float64)
        Gw[:cnt, :d] = torch.from_numpy(G_own)
        exchange_halo(Gw, lay, rank, s)
        got = Gw.numpy()[:, :d]
        for t in range(s):                                # the halo holds the next s groups, in cyclic order
            assert np.array_equal(got[cnt + t], G_all[(lo + cnt + t) % n])
        coded_want = orc.encode(B, G_all)
        a = orc.decode_vector(B, S)
        part = np.zeros(d)
        for r in range(cnt):                              # the workers that start in this rank's block
            i = lo + r
            x_i = sum(B[i, (i + t) % n] * got[r + t] for t in range(s + 1))
            assert np.allclose(x_i, coded_want[i], rtol=1e-12, atol=1e-12)
            part += a[i] * x_i
        tot = torch.from_numpy(part.copy())
        dist.all_reduce(tot)                              # the ONE collective of the data path
        worst = max(worst, float(np.linalg.norm(tot.numpy() - g_full) / np.linalg.norm(g_full)))
    dist.barrier()
    torch.save({"worst": worst}, os.path.join(out, f"s{rank}.pt"))
    dist.destroy_process_group()


def test_sharded_step_halo_and_sum_recover_the_full_gradient(tmp_path):
    """Section II-C over two ranks: contiguous blocks of partitions, the halo of s partial gradients from the ring
    neighbour, the local shares of the decode summed by one all-reduce.  Arithmetic by the oracle (this is a test
    of the partitioning, of the exchange and of the sum, on CPU)."""
    port = _free_port()
    mp.spawn(_shard_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        assert torch.load(tmp_path / f"s{r}.pt")["worst"] < 1e-9
