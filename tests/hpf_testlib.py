"""Helpers shared by the GPU parity tests: bind a model on torch memory, read tensors back, rel-L2."""
import numpy as np
import torch

import paper_1911_05146_b200 as hpf
import workloads as wl

TOL_TENSOR = 1e-2     # relative L2 per activation and gradient tensor
TOL_LOSS = 1e-3       # relative, on the loss
# The judge of every comparison is the PLAIN oracle: it takes nothing from the GPU.  The gradient is a discontinuous
# function of the forward values (the derivative of ReLU is a step), so an implementation whose pre-activation z
# differs from the oracle's by a rounding error takes the other branch where |z| is below that error, and a handful
# of such flips per tensor can add up, through a thousand layers, to more than the tolerance.  Only for a backward
# tensor that misses the tolerance against the plain oracle is a second, diagnostic oracle run consulted, in which
# the oracle evaluates its gradient under the decisions z > 0 the GPU took - and only inside the window
# |z| < TAU*|gamma| (a GPU decision that differs outside it fails the test), and only if those decisions are a
# vanishing fraction of all decisions.  The window follows the forward accuracy of the convolution path: for the
# fp32-class paths (three-pass TF32, CUDA cores) it is ten times the worst relative L2 error of an activation tensor
# measured at full depth (3.1e-5 on ResNet-1001; a single element's error exceeds the tensor's rms error by a few times,
# and at 1e-4 two of 3.5e8 decisions of the wide ResNet-1001 fell outside).
TAU = 3e-4
TAU_ONE_PASS = 0.02
MAX_DECISION_FRACTION = 2e-5          # of all ReLU decisions of the micro-batch (fp32-class paths)
MAX_DECISION_FRACTION_ONE_PASS = 5e-3

PARITY_LOG = []       # one line per compared step; the test session prints them in its summary


def rel_l2(a, ref):
    a = np.asarray(a, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.linalg.norm(ref)
    if den == 0.0:
        return 0.0 if np.linalg.norm(a) == 0.0 else np.inf
    return float(np.linalg.norm(a - ref) / den)


class Bound:
    """A model bound to torch-owned device memory."""

    def __init__(self, ops, in_hwc, B, M, cuts, theta, options=None, device="cuda:0", side_streams=True, backward_streams=False):
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
        n_streams = self.model.num_stream_slots() * (3 if backward_streams else (2 if side_streams else 1))
        self.streams = [torch.cuda.Stream(device=self.dev) for _ in range(n_streams)]
        torch.cuda.synchronize()
        self.model.bind(self.params, self.slots, self.avg, self.ws, self.streams)

    def upload(self, x, labels):
        self.x = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(self.dev)
        self.labels = torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).to(self.dev)
        torch.cuda.synchronize()

    def step(self, one_graph=False):
        if one_graph:
            self.model.forward_backward(self.x, self.labels)
        else:
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
    """DIAGNOSTIC: the oracle's micro-batch m evaluated under the GPU's in-window ReLU decisions; fails on any
    decision the forward tolerance does not leave open.  Never the first judge of a comparison (see compare_microbatch)."""
    from oracle import reference as ora
    b = bd.B // bd.M
    dec = {i: (bd.tensor(i, m) > 0).astype(np.uint8) for i, o in enumerate(bd.ops) if o.kind in (wl.BNRELU, wl.RELU)}
    r = ora.microbatch(bd.ops, bd.in_hwc, theta, x[m * b:(m + 1) * b], labels[m * b:(m + 1) * b], cuts=cuts, want=want,
                       decisions=dec, tau=tau)
    assert r["decision_violations"] == 0, r["decision_violations"]
    r["decisions_total"] = int(sum(d.size for d in dec.values()))
    return r


def _tensor_errors(bd, m, slots, offs, r, tensors):
    """rel-L2 of every stored activation, every activation gradient and every parameter-gradient tensor of
    micro-batch m against oracle result r."""
    err = {}
    if tensors:
        for i in range(len(bd.ops)):
            a = bd.tensor_or_none(i, m)          # None: a convolution whose output lives only inside the fused residual add
            if a is not None:
                err[("act", i)] = rel_l2(a, r["act"][i])
            err[("dact", i)] = rel_l2(bd.tensor(i, m, grad=True), r["dact"][i])
    for i, (w_off, w_cnt, b_off, b_cnt) in enumerate(offs):
        for which, off, cnt in (("w", w_off, w_cnt), ("b", b_off, b_cnt)):
            if cnt:
                err[("g", i, which)] = rel_l2(slots[m, off:off + cnt], r["g"][off:off + cnt])
    return err


def compare_microbatch(bd, m, theta, x, labels, slots, offs, loss_m, cuts=None, tau=TAU, max_fraction=MAX_DECISION_FRACTION,
                       tensors=True, diagnostic=True, skip=()):
    """Micro-batch m of the GPU step against the oracle.

    1. The plain oracle (no input from the GPU) judges the loss, every activation, and every gradient tensor.
    `skip`: keys of tensors left out (a gradient that is zero analytically has no relative error to speak of).
    2. A gradient tensor beyond the tolerance there is named, and must then hold the tolerance against the oracle
       evaluated under the GPU's in-window ReLU decisions, with no decision outside the window and at most
       max(8, max_fraction * decisions) decisions taken from the GPU.
    Returns the worst figures of both comparisons (the second one is also run when nothing failed, as a diagnostic,
    unless diagnostic=False)."""
    from oracle import reference as ora
    b = bd.B // bd.M
    plain = ora.microbatch(bd.ops, bd.in_hwc, theta, x[m * b:(m + 1) * b], labels[m * b:(m + 1) * b], cuts=cuts,
                           want=None if tensors else [])
    assert abs(loss_m - plain["loss"]) <= TOL_LOSS * abs(plain["loss"]), ("loss", m, loss_m, plain["loss"])
    e_plain = {k: e for k, e in _tensor_errors(bd, m, slots, offs, plain, tensors).items() if k not in skip}
    for k, e in e_plain.items():
        if k[0] == "act":
            assert e <= TOL_TENSOR, (k, m, e)          # forward values are continuous: the plain oracle alone decides
    over = {k: e for k, e in e_plain.items() if k[0] != "act" and not e <= TOL_TENSOR}
    out = {"m": m, "plain": {kind: max([e for k, e in e_plain.items() if k[0] == kind] or [0.0]) for kind in ("act", "dact", "g")},
           "over": over, "matched": None, "decisions_used": None, "decisions_total": None, "plain_result": plain}
    if over or diagnostic:
        r = matched_oracle(bd, m, theta, x, labels, cuts=cuts, want=None if tensors else [], tau=tau)
        e_m = _tensor_errors(bd, m, slots, offs, r, tensors)
        out["matched"] = {kind: max([e for k, e in e_m.items() if k[0] == kind] or [0.0]) for kind in ("act", "dact", "g")}
        out["decisions_used"], out["decisions_total"] = int(r["decisions_used"]), r["decisions_total"]
        out["matched_result"] = r
        for k in over:
            assert e_m[k] <= TOL_TENSOR, ("beyond the tolerance against the plain oracle AND under matched decisions", k, m, over[k], e_m[k])
        if over:
            allowed = max(8, int(max_fraction * r["decisions_total"]))
            assert r["decisions_used"] <= allowed, ("too many ReLU decisions taken from the GPU", r["decisions_used"], allowed)
    return out


def log_parity(name, results):
    """One summary line for the comparisons of a test (printed at the end of the test session)."""
    worst_p = {k: max(r["plain"][k] for r in results) for k in ("act", "dact", "g")}
    have_m = [r for r in results if r["matched"] is not None]
    worst_m = {k: max(r["matched"][k] for r in have_m) for k in ("act", "dact", "g")} if have_m else None
    over = sorted({k for r in results for k in r["over"]})
    over_worst = max([e for r in results for e in r["over"].values()] or [0.0])
    used = sum(r["decisions_used"] or 0 for r in results)
    total = sum(r["decisions_total"] or 0 for r in results)
    line = ("%s: micro-batches %s | plain oracle worst rel-L2 act %.2e dact %.2e g %.2e | " %
            (name, [r["m"] for r in results], worst_p["act"], worst_p["dact"], worst_p["g"]))
    if worst_m:
        line += "GPU-decision oracle (diagnostic) worst dact %.2e g %.2e, decisions_used %d of %d | " % (worst_m["dact"], worst_m["g"], used, total)
    line += ("every tensor within %.0e of the plain oracle" % TOL_TENSOR) if not over else \
            ("%d gradient tensors beyond %.0e against the plain oracle (worst %.2e, first %s): judged under GPU decisions" %
             (len(over), TOL_TENSOR, over_worst, over[:4]))
    PARITY_LOG.append(line)
    print(line)
    return line
