"""Micro-batch count tuner (Section 5.3, pipelining paragraph: the number of pipeline stages ranges from 1 to the
batch size; the suggested search starts at the batch size and halves it).

`halving_candidates` is the search order; `tune_microbatches` times one training step per candidate through the
library on the current CUDA device and returns the fastest.  The count changes the arithmetic (batch-norm
statistics are per micro-batch), so the caller decides whether the tuned value is admissible for its experiment.
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


def time_step(ops, in_shape, cuts, n_microbatches, params, steps=3, warmup=2, device=None):
    """Milliseconds per forward+backward+average step with `n_microbatches` micro-batches (CUDA events)."""
    dev = torch.device(device if device is not None else "cuda:%d" % torch.cuda.current_device())
    model = _b.Model(ops, in_shape, cuts, n_microbatches)
    try:
        G = model.num_params()
        theta = params.to(dev, torch.float32)
        slots = torch.empty((n_microbatches, G), device=dev)
        avg = torch.empty(G, device=dev)
        ws = torch.empty(model.workspace_bytes(), dtype=torch.uint8, device=dev)
        streams = [torch.cuda.Stream(device=dev) for _ in range(2 * model.num_partitions())]
        x = torch.randn(tuple(in_shape), device=dev)
        labels = torch.zeros(in_shape[0], dtype=torch.int32, device=dev)
        torch.cuda.synchronize(dev)
        model.bind(theta, slots, avg, ws, streams)
        s0 = streams[0]

        def step():
            model.forward(x, labels); model.backward(); model.grad_average()
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
        return e0.elapsed_time(e1) / steps
    finally:
        model.close()


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
