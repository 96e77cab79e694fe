"""Hybrid parallelism on several GPUs: partitions on different GPUs, replicas of the whole pipeline side by side
(Section 5.3: one process per model-partition, send / recv of activations and partial errors between neighbouring
partitions, one allreduce communicator per model-partition across the replicas; Section 6.5 runs it at scale).

Every rank binds the SAME model (op list, cuts, micro-batch count), so every rank has the same memory plan, and runs only
the cells of the partition it owns (`Model.forward_cell` / `backward_cell`).  A tensor that crosses a cut lives at the same
workspace offset on both sides: the hand-off is a copy from the producer's workspace into the consumer's own memory
(`torch.distributed` send / recv over NCCL, or a device copy in the one-process emulation) - never a load from a peer's
memory inside a kernel.  After the backward pass each rank averages its micro-batch gradient slots and the ranks that own
the same partition average that partition's slice of the gradient over the replicas (`all_reduce` on that partition's
group).

    rank = replica * P + partition

`run_step` is one rank's step.  `emulate_step` runs all ranks of a layout in ONE process on one GPU, cell by cell in
pipeline order with device copies for the hand-offs: what the tests use where only one GPU is at hand.
"""
import torch

from . import binding as _b


class HybridLayout:
    """Which rank owns which (replica, partition), and who talks to whom."""

    def __init__(self, world_size, n_partitions):
        if n_partitions < 1 or world_size < 1 or world_size % n_partitions:
            raise ValueError("the world size must be a multiple of the partition count")
        self.world, self.P, self.R = int(world_size), int(n_partitions), int(world_size) // int(n_partitions)

    def coords(self, rank):
        if not 0 <= rank < self.world:
            raise ValueError("rank out of range")
        return divmod(int(rank), self.P)                 # (replica, partition)

    def rank_of(self, replica, partition):
        if not (0 <= replica < self.R and 0 <= partition < self.P):
            raise ValueError("coordinates out of range")
        return replica * self.P + partition

    def partition_group(self, partition):
        """Ranks that own `partition`, one per replica: the members of that partition's allreduce communicator."""
        return [self.rank_of(r, partition) for r in range(self.R)]

    def below(self, rank):
        r, p = self.coords(rank)
        return self.rank_of(r, p - 1) if p > 0 else None

    def above(self, rank):
        r, p = self.coords(rank)
        return self.rank_of(r, p + 1) if p < self.P - 1 else None


class StagePlan:
    """What the owner of partition p receives and sends, from the model's bookkeeping tables (host only)."""

    def __init__(self, model, p):
        P = model.num_partitions()
        self.p, self.P = p, P
        live = lambda cut: [model.boundary_desc(cut, i) for i in range(model.boundary_count(cut))]
        self.fwd_recv = live(p - 1) if p > 0 else []                 # (op, (b, H, W, C)) activations from below
        self.fwd_send = live(p) if p < P - 1 else []
        self.bwd_recv = model.backward_messages(p) if p < P - 1 else []      # gradient buffers handed down from above
        self.bwd_send = model.backward_messages(p - 1) if p > 0 else []
        self.param_first, self.param_count = model.partition_param_range(p)


class Stage:
    """One rank: the model bound on this rank's GPU, running the cells of partition p only."""

    def __init__(self, ops, in_shape, cuts, n_microbatches, theta, p, device, options=None):
        self.dev = torch.device(device)
        self.p, self.M = p, n_microbatches
        self.model = _b.Model(ops, in_shape, cuts, n_microbatches)
        self.model.set_option(_b.OPT_GRAPH, 0)                       # cells are enqueued directly
        for k, v in (options or {}).items():
            self.model.set_option(k, v)
        self.P = self.model.num_partitions()
        self.plan = StagePlan(self.model, p)
        G = self.model.num_params()
        with torch.cuda.device(self.dev):
            self.params = theta.to(self.dev, torch.float32).contiguous()
            self.slots = torch.zeros((n_microbatches, G), device=self.dev)
            self.avg = torch.zeros(G, device=self.dev)
            self.ws = torch.empty(self.model.workspace_bytes(), dtype=torch.uint8, device=self.dev)
            self.streams = [torch.cuda.Stream(device=self.dev) for _ in range(2 * self.model.num_stream_slots())]
            torch.cuda.synchronize(self.dev)
            self.model.bind(self.params, self.slots, self.avg, self.ws, self.streams)
        self.stream = self.streams[p]
        self.x = self.labels = None

    def _view(self, op, m, grad):
        ptr, shape = self.model.tensor_ptr(op, m, grad)
        off = ptr - self.ws.data_ptr()
        n = 1
        for d in shape:
            n *= d
        return self.ws[off:off + 4 * n].view(torch.float32).view(shape)

    def act(self, op, m):
        return self._view(op, m, False)

    def grad(self, op, m):
        return self._view(op, m, True)

    def begin(self, x=None, labels=None):
        self.x, self.labels = x, labels
        self.model.prepare_partition(self.p)

    def forward(self, m):
        self.model.forward_cell(self.p, m, self.x if self.p == 0 else None, self.labels if self.p == self.P - 1 else None)

    def backward(self, m):
        self.model.backward_cell(self.p, m)

    def finish(self):
        """Joins the weight-gradient stream, averages the micro-batch slots; returns this partition's slice of the average."""
        self.model.join_partition(self.p)
        self.stream.synchronize()
        self.model.grad_average()                                    # the library's kernel, over the whole flat buffer
        self.model.synchronize(0)
        a, n = self.plan.param_first, self.plan.param_count
        return self.avg[a:a + n]

    def losses(self):
        ptr = self.model.loss_slots_ptr()
        off = ptr - self.ws.data_ptr()
        return self.ws[off:off + 4 * self.M].view(torch.float32)

    def sync(self):
        self.stream.synchronize()


class TorchDistComm:
    """send / recv / per-partition allreduce on torch.distributed (NCCL between GPUs; gloo in the CPU tests).  One process
    group per partition, created once: the paper's one communicator per model-partition."""

    def __init__(self, layout, rank):
        import torch.distributed as dist
        self.dist, self.layout, self.rank = dist, layout, rank
        self.groups = {}
        for p in range(layout.P):                                    # every rank creates every group, in the same order
            ranks = layout.partition_group(p)
            self.groups[p] = dist.new_group(ranks) if len(ranks) > 1 else None

    def send(self, tensor, dst):
        # the caller has waited for the producing kernels; the copy engine / NCCL reads a finished tensor
        self.dist.send(tensor.contiguous(), dst)

    def recv(self, tensor, src):
        self.dist.recv(tensor, src)
        if tensor.is_cuda:
            # NCCL completes on its own stream: the cell that reads the tensor is enqueued on the stage's stream only
            # after the data has landed
            torch.cuda.current_stream(tensor.device).synchronize()

    def all_reduce_mean(self, tensor, partition):
        g = self.groups[partition]
        if g is None:
            return
        if self.dist.get_backend(g) == "nccl":
            self.dist.all_reduce(tensor, op=self.dist.ReduceOp.AVG, group=g)     # the average happens inside the collective
        else:
            self.dist.all_reduce(tensor, op=self.dist.ReduceOp.SUM, group=g)     # gloo (CPU tests) has no averaging reduction
            tensor /= self.layout.R


class SingleRankComm:
    """The communicator of a world of one rank: nothing to send, nothing to average."""

    def send(self, tensor, dst):
        raise RuntimeError("a single rank has no neighbour")

    def recv(self, tensor, src):
        raise RuntimeError("a single rank has no neighbour")

    def all_reduce_mean(self, tensor, partition):
        pass


def run_step(stage, layout, rank, comm, x=None, labels=None):
    """One rank's step.  `stage` owns partition layout.coords(rank)[1]; x / labels: this replica's batch (used by the first /
    last partition).  Forward: for every micro-batch, receive the live set from below, run the cell, send the live set up.
    Backward: receive the gradient buffers from above, run the cell, send down.  Messages of one cut go in the tables' order
    on both sides, and data flows one way per phase, so the blocking calls cannot wait on each other in a cycle.  Returns
    this partition's slice of the gradient, averaged over micro-batches and replicas."""
    _, p = layout.coords(rank)
    lo, hi = layout.below(rank), layout.above(rank)
    plan = stage.plan
    stage.begin(x, labels)
    for m in range(stage.M):
        for op, _ in plan.fwd_recv:
            comm.recv(stage.act(op, m), lo)
        stage.forward(m)
        if plan.fwd_send:
            stage.sync()                                              # the cell's kernels are done before its output leaves
            for op, _ in plan.fwd_send:
                comm.send(stage.act(op, m), hi)
    for m in range(stage.M):
        for op, _ in plan.bwd_recv:
            comm.recv(stage.grad(op, m), hi)
        stage.backward(m)
        if plan.bwd_send:
            stage.sync()
            for op, _ in plan.bwd_send:
                comm.send(stage.grad(op, m), lo)
    g = stage.finish()
    comm.all_reduce_mean(g, p)
    return g


def emulate_step(stages, layout, batches):
    """All ranks of `layout` in one process: stages[rank], batches[replica] = (x, labels) device tensors.  Cells run in
    pipeline tick order, hand-offs are device copies between the stages' workspaces, the per-partition allreduce is a mean
    over the replicas' slices.  Returns {rank: averaged gradient slice}."""
    P, R = layout.P, layout.R
    M = stages[0].M
    for rank, st in enumerate(stages):
        r, p = layout.coords(rank)
        st.begin(*batches[r])
    for t in range(P + M - 1):
        for r in range(R):
            for p in range(P):
                m = t - p
                if not 0 <= m < M:
                    continue
                st = stages[layout.rank_of(r, p)]
                if p > 0:
                    src = stages[layout.rank_of(r, p - 1)]
                    src.sync()
                    for op, _ in st.plan.fwd_recv:
                        st.act(op, m).copy_(src.act(op, m))
                    torch.cuda.synchronize()
                st.forward(m)
    for t in range(P + M - 1):
        for r in range(R):
            for p in range(P - 1, -1, -1):
                m = t - (P - 1 - p)
                if not 0 <= m < M:
                    continue
                st = stages[layout.rank_of(r, p)]
                if p < P - 1:
                    src = stages[layout.rank_of(r, p + 1)]
                    src.sync()
                    for op, _ in st.plan.bwd_recv:
                        st.grad(op, m).copy_(src.grad(op, m))
                    torch.cuda.synchronize()
                st.backward(m)
    slices = {rank: st.finish() for rank, st in enumerate(stages)}
    for p in range(P):
        group = layout.partition_group(p)
        mean = slices[group[0]].clone()
        for rank in group[1:]:
            mean += slices[rank]
        mean /= R
        for rank in group:
            slices[rank].copy_(mean)
    return slices
