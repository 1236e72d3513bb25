"""One nested-gradient-code problem sharded over several GPUs, one process per GPU.

The method's own setting is a set of independent workers, each holding a few data partitions (Section II-C).
Here rank r holds a contiguous block of the n partition groups and simulates the workers whose windows start
in that block.  Per iteration:

  1. every rank computes the partial gradients g_j of its own groups              (ngc_shard_gradients)
  2. worker i needs g_i .. g_{i+s} (cyclic): the s groups behind a rank's block are fetched from the ranks
     that own them                                                               (exchange_halo, point to point)
  3. every rank encodes its workers and forms its share sum_{i in S, i mine} a_i x_i of the decode
                                                                                  (ngc_shard_encode_decode)
  4. one all-reduce (sum) of l values gives the decoded gradient                  (torch.distributed)

The stopping rule runs on every rank on the same task times, so all ranks agree on the component code and
on the responsive set without talking.  `ShardLayout` and `exchange_halo` are plain index logic and
torch.distributed calls on whatever device the tensors live on; the arithmetic is the library's kernels.
No TMA multicast, no peer-memory operands: the exchange is NCCL send / receive and all-reduce.
"""
from __future__ import annotations

import json
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class ShardLayout:
    """Contiguous blocks of the n partition groups (= workers), one per rank."""
    n: int
    world: int

    def first(self, rank: int) -> int:
        return rank * self.n // self.world

    def count(self, rank: int) -> int:
        return self.first(rank + 1) - self.first(rank)

    def owner(self, group: int) -> int:
        """Rank whose block contains `group`."""
        group %= self.n
        return ((group + 1) * self.world - 1) // self.n

    def halo(self, rank: int, s: int):
        """Where the s groups behind rank's block come from, in window order:
        a list of (source rank, first local row at the source, number of rows, first halo row here)."""
        out = []
        g = self.first(rank) + self.count(rank)
        left, row = s, 0
        while left > 0:
            g %= self.n
            src = self.owner(g)
            take = min(left, self.first(src) + self.count(src) - g)
            out.append((src, g - self.first(src), take, row))
            g += take
            row += take
            left -= take
        return out

    def sends(self, rank: int, s: int):
        """What `rank` owes the others: a list of (destination rank, first local row, number of rows)."""
        out = []
        for dst in range(self.world):
            if dst == rank:
                continue
            for src, lrow, take, _ in self.halo(dst, s):
                if src == rank:
                    out.append((dst, lrow, take))
        return out


def exchange_halo(G_window: torch.Tensor, layout: ShardLayout, rank: int, s: int, group=None) -> None:
    """Fills rows n_local .. n_local + s - 1 of G_window ([>= n_local + s][ld], rows 0 .. n_local - 1 = this rank's
    own partial gradients) with the partial gradients of the next s groups in cyclic order."""
    n_local = layout.count(rank)
    ops, keep = [], []
    for src, lrow, take, hrow in layout.halo(rank, s):
        dst_rows = G_window[n_local + hrow: n_local + hrow + take]
        if src == rank:
            dst_rows.copy_(G_window[lrow: lrow + take])       # the window wraps into this rank's own block
        else:
            ops.append(dist.P2POp(dist.irecv, dst_rows, src, group))
    for dst, lrow, take in layout.sends(rank, s):
        buf = G_window[lrow: lrow + take]
        keep.append(buf)
        ops.append(dist.P2POp(dist.isend, buf, dst, group))
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()


class ShardedStep:
    """One rank's part of the sharded iteration on its GPU (see the module text)."""

    def __init__(self, ngc, workload, X_local, y_local, rank: int, world: int, device):
        self.ngc = ngc
        self.w = workload
        self.rank, self.world = rank, world
        self.layout = ShardLayout(workload.n, world)
        self.first, self.n_local = self.layout.first(rank), self.layout.count(rank)
        self.X, self.y = X_local, y_local
        self.m = ngc.Model.make(workload.kind, workload.x_dtype, workload.rows, workload.d, workload.n_classes,
                                workload.hidden)
        self.plan = ngc.Plan(workload.n, workload.levels, seed=workload.seed)
        self.l = workload.n_params
        self.ld = (self.l + 3) // 4 * 4
        s_max = workload.levels[-1]
        self.f64 = self.plan.coded_dtype(self.m) == ngc.NGC_F64
        cdt = torch.float64 if self.f64 else torch.float32
        self.G = torch.zeros((self.n_local + s_max, self.ld), dtype=torch.float32, device=device)
        self.coded = torch.empty((self.n_local + s_max, self.l), dtype=cdt, device=device)
        self.partial = torch.empty(self.l, dtype=cdt, device=device)
        self.grad = torch.empty(self.l, dtype=torch.float32, device=device)
        # the rank's data does not change between iterations (Section II-C): derive what depends on it alone once
        self.plan.shard_prepare_data(self.m, self.X, self.n_local, torch.cuda.current_stream().cuda_stream)

    def step(self, theta, task_times, group=None):
        """Returns the stopping rule's result; self.grad holds the decoded gradient on every rank."""
        info = self.plan.select(task_times)                    # same on every rank
        s = info.sigma
        stream = torch.cuda.current_stream().cuda_stream
        self.plan.shard_gradients(self.m, theta, self.X, self.y, self.n_local, self.G, self.ld, stream)
        if self.world > 1 or s > 0:
            exchange_halo(self.G, self.layout, self.rank, s, group)
        self.plan.shard_encode_decode(self.m, info.layer, self.first, self.n_local, self.G, self.ld,
                                      info.responsive(), self.coded, self.partial, stream)
        if self.world > 1:
            dist.all_reduce(self.partial, op=dist.ReduceOp.SUM, group=group)
        self.grad.copy_(self.partial)                          # rounded to fp32 after the sum over the ranks
        return info


def bench_sharded(args, rank, local_rank, world, dev):
    """`bench.py --sharded`: the named workload as ONE problem over all ranks (strong scaling)."""
    import ngc_inputs
    import paper_2212_08580_b200 as ngc
    from bench import METRIC, UNIT, decodable_patterns, rank_max, rank_sum

    w = ngc_inputs.WORKLOADS[args.workload]
    if args.rows:
        w = ngc_inputs.shrink(w, rows=args.rows)
    layout = ShardLayout(w.n, world)
    X, y, theta = ngc_inputs.make_data(w, dev)                 # same seed everywhere: every rank draws the same data
    lo, cnt = layout.first(rank), layout.count(rank)
    Xl, yl = X[lo: lo + cnt].contiguous(), y[lo: lo + cnt].contiguous()
    del X, y
    torch.cuda.empty_cache()
    st = ShardedStep(ngc, w, Xl, yl, rank, world, dev)

    def decodable(t):
        try:
            st.plan.select(t)
            return True
        except ngc.NgcError:
            return False

    pats, skipped = decodable_patterns(w, w.levels, args.warmup + args.steps, decodable)
    for i in range(args.warmup):
        st.step(theta, pats[i])
    torch.cuda.synchronize()
    launches0 = st.plan.launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        st.step(theta, pats[args.warmup + i])
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms_total = rank_max(e0.elapsed_time(e1), world, dev)
    launches = st.plan.launch_count() - launches0
    line = {
        "metric": METRIC, "value": args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None,
        "dtype": "f32" if w.kind in ("lsq", "logistic") else "bf16", "data": "synthetic",
        "config": {"workload": w.name, "n_workers": w.n, "levels": list(w.levels), "kind": w.kind,
                   "rows_per_partition": w.rows, "d": w.d, "x_dtype": w.x_dtype,
                   "parallelism": f"one problem, partition groups in {world} contiguous blocks; halo of s partial "
                                  "gradients by send / receive, one all-reduce of the decoded gradient",
                   "l2": "inputs larger than L2" if Xl.numel() * Xl.element_size() > 126e6 else
                         "this rank's data fit in L2",
                   "undecodable_skipped": skipped},
        "gpu_launches": int(rank_sum(launches, world, dev)),
        "e2e": None, "roofline": None,
    }
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
