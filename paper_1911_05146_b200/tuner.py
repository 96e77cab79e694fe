"""Micro-batch count tuner (Section 5.3, pipelining paragraph: the number of pipeline stages ranges from 1 to the
batch size; the suggested search starts at the batch size and halves it).

`halving_candidates` is the search order; `tune_microbatches` times one training step per candidate through the
library on the current CUDA device and returns the fastest.  The count changes the arithmetic (batch-norm
statistics are per micro-batch), so the caller decides whether the tuned value is admissible for its experiment.

Load balancer by measurement (Section 5.4 names the component and leaves it open): `balance_by_measurement` runs the
pipeline, reads how long every (partition, micro-batch) cell really took while the other stages were running
(`hpf_cell_times`), apportions each partition's measured time to its ops in proportion to their modelled cost, asks
`hpf_balance_cuts` for the cuts that even out those costs, and repeats; the fastest cut list seen wins.  Cuts change
nothing in the arithmetic (the oracle's partition-count invariance), only which stage runs what.
"""
import torch

from . import binding as _b


def halving_candidates(batch, smallest=1):
    """batch, batch/2, batch/4, ... down to `smallest`, keeping the values that divide the batch."""
    out, m = [], int(batch)
    while m >= max(1, smallest):
        if batch % m == 0:
            out.append(m)
        if m == 1:
            break
        m //= 2
    return out


def time_step(ops, in_shape, cuts, n_microbatches, params, steps=3, warmup=2, device=None, cell_times=False, options=None):
    """Milliseconds per forward+backward+average step with `n_microbatches` micro-batches (CUDA events).  With
    cell_times: returns (ms, forward cells, backward cells), the cells as [partition][micro-batch] (start ns, end ns) of
    the last step."""
    dev = torch.device(device if device is not None else "cuda:%d" % torch.cuda.current_device())
    model = _b.Model(ops, in_shape, cuts, n_microbatches)
    try:
        for k, v in (options or {}).items():
            model.set_option(k, v)
        if cell_times:
            model.set_option(_b.OPT_CELL_TIMES, 1)
        G = model.num_params()
        theta = params.to(dev, torch.float32)
        slots = torch.empty((n_microbatches, G), device=dev)
        avg = torch.empty(G, device=dev)
        ws = torch.empty(model.workspace_bytes(), dtype=torch.uint8, device=dev)
        streams = [torch.cuda.Stream(device=dev) for _ in range(3 * model.num_stream_slots())]      # stage, weight-gradient, backward
        x = torch.randn(tuple(in_shape), device=dev)
        labels = torch.zeros(in_shape[0], dtype=torch.int32, device=dev)
        torch.cuda.synchronize(dev)
        model.bind(theta, slots, avg, ws, streams)
        s0 = streams[0]

        def step():
            model.forward_backward(x, labels); model.grad_average()
        for _ in range(warmup):
            step()
        model.synchronize(0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s0)
        for _ in range(steps):
            step()
        e1.record(s0)
        model.synchronize(0)
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / steps
        if cell_times:
            return ms, model.cell_times(0), model.cell_times(1)
        return ms
    finally:
        model.close()


def partition_times_us(cells_fwd, cells_bwd):
    """Mean time (microseconds) a partition's cells took, forward plus backward, as the pipeline ran them."""
    out = []
    for f, b in zip(cells_fwd, cells_bwd):
        tf = sum(e - s for s, e in f) / len(f)
        tb = sum(e - s for s, e in b) / len(b)
        out.append((tf + tb) / 1e3)
    return out


def balance_by_measurement(ops, in_shape, n_partitions, n_microbatches, params, start_cuts, rounds=3, steps=3, options=None):
    """Cuts chosen from what the pipeline measures.  Returns (best_cuts, history) with history a list of
    {"cuts", "ms", "partition_us"}; history[0] is the start (e.g. equal op counts)."""
    b = in_shape[0] // n_microbatches
    cost = _b.estimate_op_costs(ops, (b,) + tuple(in_shape[1:]))
    cost = [max(c, 1e-3) for c in cost]                    # an op the model prices at zero still belongs to some partition
    cuts = list(start_cuts)
    history = []
    for r in range(rounds + 1):
        ms, cf, cb = time_step(ops, in_shape, cuts, n_microbatches, params, steps=steps, cell_times=True, options=options)
        part_us = partition_times_us(cf, cb)
        history.append({"cuts": list(cuts), "ms": ms, "partition_us": part_us})
        if r == rounds:
            break
        # apportion each partition's measured time to its ops by modelled cost
        bounds = [0] + list(cuts) + [len(ops)]
        for p in range(n_partitions):
            lo, hi = bounds[p], bounds[p + 1]
            modelled = sum(cost[lo:hi])
            scale = part_us[p] / modelled if modelled > 0 else 1.0
            for i in range(lo, hi):
                cost[i] *= scale
        new_cuts = _b.balance_cuts(cost, n_partitions)
        if new_cuts == cuts:
            break
        cuts = new_cuts
    best = min(history, key=lambda h: h["ms"])
    return best["cuts"], history


def tune_microbatches(ops, in_shape, cuts, params, smallest_microbatch=1, largest_count=None, patience=1, steps=3):
    """Walks the halving sequence from the largest admissible count downwards and stops once `patience` successive
    candidates were slower than the best so far.  Returns (best_count, {count: ms})."""
    batch = int(in_shape[0])
    tried = {}
    best, worse = None, 0
    for m in halving_candidates(batch):
        if batch // m < smallest_microbatch or (largest_count is not None and m > largest_count):
            continue
        tried[m] = time_step(ops, in_shape, cuts, m, params, steps=steps)
        if best is None or tried[m] < tried[best]:
            best, worse = m, 0
        else:
            worse += 1
            if worse > patience:
                break
    return best, tried
