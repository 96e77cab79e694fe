"""Worker of tests/test_hybrid_cpu.py: one gloo rank of a hybrid-parallel step with the compute replaced by a stand-in.

The layout, the per-partition message tables (from the library's host-side bookkeeping), the send / recv order and the
per-partition allreduce groups are the real ones (paper_1911_05146_b200.hybrid); only the cells are faked: a stand-in
"stage" fills what it sends with numbers that encode (partition, micro-batch, position), so the receiving side can check
that every message arrived where and when the tables say.
"""
import json
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import workloads as wl  # noqa: E402
import paper_1911_05146_b200 as hpf  # noqa: E402
from paper_1911_05146_b200.hybrid import HybridLayout, StagePlan, TorchDistComm, run_step  # noqa: E402


def code(kind, p, m, j):
    return float(100000 * kind + 1000 * p + 10 * m + j)


class FakeStage:
    """The interface run_step uses, on CPU tensors."""

    def __init__(self, model, p, M):
        self.p, self.M, self.plan = p, M, StagePlan(model, p)
        self.buf, self.log, self.events = {}, [], []

    def _t(self, op, m, grad, shape):
        key = (op, m, grad)
        if key not in self.buf:
            self.buf[key] = torch.full(shape, -1.0)
        return self.buf[key]

    def act(self, op, m):
        shape = dict(self.plan.fwd_recv + self.plan.fwd_send)[op]
        return self._t(op, m, False, shape)

    def grad(self, op, m):
        shape = dict(self.plan.bwd_recv + self.plan.bwd_send)[op]
        return self._t(op, m, True, shape)

    def begin(self, x=None, labels=None):
        self.events.append("begin")

    def forward(self, m):
        self.log.append(("fwd", m, [float(self.act(op, m).flatten()[0]) for op, _ in self.plan.fwd_recv],
                         [bool((self.act(op, m) == self.act(op, m).flatten()[0]).all()) for op, _ in self.plan.fwd_recv]))
        for j, (op, _) in enumerate(self.plan.fwd_send):
            self.act(op, m).fill_(code(1, self.p, m, j))

    def backward(self, m):
        self.log.append(("bwd", m, [float(self.grad(op, m).flatten()[0]) for op, _ in self.plan.bwd_recv],
                         [bool((self.grad(op, m) == self.grad(op, m).flatten()[0]).all()) for op, _ in self.plan.bwd_recv]))
        for j, (op, _) in enumerate(self.plan.bwd_send):
            self.grad(op, m).fill_(code(2, self.p, m, j))

    def sync(self):
        pass

    def finish(self):
        return torch.full((self.plan.param_count,), float(self.rank_value))


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    P = int(sys.argv[1])
    dist.init_process_group("gloo")
    ops = wl.resnet_v2_cifar(1)
    B, M = 4, 2
    cuts = [12] if P == 2 else []                 # mid-block: two tensors cross, and a residual add's gradient is pending
    model = hpf.Model(ops, (B, 32, 32, 3), cuts, M)
    layout = HybridLayout(world, P)
    r, p = layout.coords(rank)
    stage = FakeStage(model, p, M)
    stage.rank_value = rank + 1
    comm = TorchDistComm(layout, rank)
    g = run_step(stage, layout, rank, comm)
    gathered = [None] * world
    dist.all_gather_object(gathered, {"coords": (r, p), "log": stage.log, "g0": float(g[0]), "g_all_equal": bool((g == g[0]).all()),
                                      "count": int(g.numel()), "fwd_send": [op for op, _ in stage.plan.fwd_send],
                                      "fwd_recv": [op for op, _ in stage.plan.fwd_recv], "bwd_send": [op for op, _ in stage.plan.bwd_send],
                                      "bwd_recv": [op for op, _ in stage.plan.bwd_recv], "group": layout.partition_group(p),
                                      "param_range": (stage.plan.param_first, stage.plan.param_count)})
    if rank == 0:
        print(json.dumps({"ranks": gathered, "G": model.num_params()}), flush=True)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
