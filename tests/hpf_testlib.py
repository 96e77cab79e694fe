"""Helpers shared by the GPU parity tests: bind a model on torch memory, read tensors back, rel-L2."""
import numpy as np
import torch

import paper_1911_05146_b200 as hpf
import workloads as wl

TOL_TENSOR = 1e-2     # relative L2 per activation and gradient tensor
TOL_LOSS = 1e-3       # relative, on the loss
# ReLU decisions: the gradient is a discontinuous function of the forward values, so both sides must take
# the decision z > 0 on the same side wherever the forward tolerance leaves it open.  The oracle keeps its own
# decision where |z| >= TAU*|gamma| (a GPU disagreement there fails the test) and evaluates the gradient under
# the GPU's decision inside that window.  The window follows the forward accuracy of the convolution path:
# fp32-class (three-pass TF32, CUDA cores) or one TF32 pass.
TAU = 2e-3
TAU_ONE_PASS = 0.02


def rel_l2(a, ref):
    a = np.asarray(a, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.linalg.norm(ref)
    if den == 0.0:
        return 0.0 if np.linalg.norm(a) == 0.0 else np.inf
    return float(np.linalg.norm(a - ref) / den)


class Bound:
    """A model bound to torch-owned device memory."""

    def __init__(self, ops, in_hwc, B, M, cuts, theta, options=None, device="cuda:0", side_streams=True):
        self.ops, self.in_hwc, self.B, self.M, self.cuts = ops, tuple(in_hwc), B, M, list(cuts)
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.model = hpf.Model(ops, (B,) + self.in_hwc, self.cuts, M)
        for k, v in (options or {}).items():
            self.model.set_option(k, v)
        self.G = self.model.num_params()
        self.params = torch.from_numpy(np.ascontiguousarray(theta, dtype=np.float32)).to(self.dev)
        self.slots = torch.full((M, self.G), float("nan"), dtype=torch.float32, device=self.dev)
        self.avg = torch.full((self.G,), float("nan"), dtype=torch.float32, device=self.dev)
        self.ws = torch.empty(self.model.workspace_bytes(), dtype=torch.uint8, device=self.dev)
        n_streams = self.model.num_partitions() * (2 if side_streams else 1)
        self.streams = [torch.cuda.Stream(device=self.dev) for _ in range(n_streams)]
        torch.cuda.synchronize()
        self.model.bind(self.params, self.slots, self.avg, self.ws, self.streams)

    def upload(self, x, labels):
        self.x = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(self.dev)
        self.labels = torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).to(self.dev)
        torch.cuda.synchronize()

    def step(self):
        self.model.forward(self.x, self.labels)
        self.model.backward()
        self.model.grad_average()
        loss = self.model.loss()
        self.model.synchronize(60000)
        return loss

    def _view(self, ptr, shape):
        off = ptr - self.ws.data_ptr()
        n = int(np.prod(shape))
        assert 0 <= off and off + 4 * n <= self.ws.numel()
        return self.ws[off:off + 4 * n].view(torch.float32).reshape(shape).cpu().numpy()

    def tensor(self, op, m, grad=False):
        ptr, shape = self.model.tensor_ptr(op, m, grad)
        return self._view(ptr, shape)

    def tensor_or_none(self, op, m):
        """The stored output of op, or None when it is a convolution fused into a residual add."""
        try:
            return self.tensor(op, m)
        except hpf.HpfError as e:
            assert e.status == -3 and self.ops[op].kind == wl.CONV, e
            return None

    def message(self, cut, i, m, grad=False):
        t, shape = self.model.boundary_desc(cut, i)
        return self._view(self.model.message_ptr(cut, i, m, grad), shape)

    def loss_slots(self):
        return self._view(self.model.loss_slots_ptr(), (self.M,))


def seeded(ops, in_hwc, B, seed=0, bn_jitter=0.0):
    x, labels = wl.draw_inputs(B, in_hwc, ops[-1].c_out, seed_x=wl.inputs.SEED_X + seed, seed_labels=wl.inputs.SEED_LABELS + seed)
    theta = wl.draw_params(ops, seed=wl.inputs.SEED_PARAMS + seed, bn_jitter=bn_jitter)
    return x, labels, theta


def matched_oracle(bd, m, theta, x, labels, cuts=None, want=None, tau=TAU):
    """The oracle's micro-batch m with the GPU's in-window ReLU decisions; fails on any decision the
    forward tolerance does not leave open."""
    from oracle import reference as ora
    b = bd.B // bd.M
    dec = {i: (bd.tensor(i, m) > 0).astype(np.uint8) for i, o in enumerate(bd.ops) if o.kind in (wl.BNRELU, wl.RELU)}
    r = ora.microbatch(bd.ops, bd.in_hwc, theta, x[m * b:(m + 1) * b], labels[m * b:(m + 1) * b], cuts=cuts, want=want,
                       decisions=dec, tau=tau)
    assert r["decision_violations"] == 0, r["decision_violations"]
    return r
