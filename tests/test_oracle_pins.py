"""Pins of the fp64 CPU oracle against what the mathematics and the paper fix.

None of these re-type the oracle's own formulas: they use finite differences of
the loss, adjoint identities, closed forms, invariances of the method
(partition count, micro-batching), a brute-force second formulation and a
library cross-check (torch CPU fp64 + autograd).
"""
import numpy as np
import pytest

import workloads as wl
from oracle import reference as ora


def tiny_cifar():
    return wl.resnet_v2_cifar(1, widths=(4, 8, 16), n_classes=5), (8, 8, 3)


def tiny_imagenet():
    return wl.resnet_v2_imagenet(blocks=(1, 1), widths=(4, 8), n_classes=7), (16, 16, 3)


def tiny_v1():
    """Post-activation basic blocks (BN without ReLU, ADD, ReLU), with a strided 3x3 and a projection shortcut."""
    return wl.resnet_v1_cifar(1, widths=(4, 8), n_classes=5), (8, 8, 3)


def tiny_vgg():
    """Convolution + ReLU groups with 2x2 max-pools and hidden fully connected layers, no batch norm."""
    return wl.vgg16_cifar(widths=(4, 8, 8), convs=(2, 1, 2), fc=12, n_classes=5), (8, 8, 3)


def _setup(builder, B, seed=0):
    ops, hwc = builder()
    x, labels = wl.draw_inputs(B, hwc, ops[-1].c_out, seed_x=100 + seed, seed_labels=200 + seed)
    theta = wl.draw_params(ops, seed=300 + seed, bn_jitter=0.3)
    return ops, hwc, x.astype(np.float64), labels, theta.astype(np.float64)


# ------------------------------------------------------------------ P1
@pytest.mark.parametrize("builder", [tiny_cifar, tiny_imagenet, tiny_v1, tiny_vgg])
def test_finite_differences_every_backward_formula(builder):
    """Central differences of the step loss against the averaged gradient: pins
    every backward formula, the BN coupling across samples and the 1/M."""
    ops, hwc, x, labels, theta = _setup(builder, B=4)
    M = 2
    base = ora.step(ops, hwc, theta, x, labels, M)
    g = base["g_avg"]
    rng = np.random.default_rng(7)
    offs, G = wl.param_offsets(ops)
    # every BN and head parameter, and a sample of the conv weights of every conv
    idx = []
    for o, (w_off, w_cnt, b_off, b_cnt) in zip(ops, offs):
        if o.kind == wl.CONV:
            idx += list(w_off + rng.choice(w_cnt, size=min(w_cnt, 12), replace=False))
        else:
            idx += list(range(w_off, w_off + min(w_cnt, 8))) + list(range(b_off, b_off + min(b_cnt, 8)))
    h = 1e-5
    bad = checked = 0
    for j in idx:
        def L(step):
            t = theta.copy(); t[j] += step
            return ora.step(ops, hwc, t, x, labels, M)["loss"]
        fd1 = (L(h) - L(-h)) / (2 * h)
        fd2 = (L(h / 2) - L(-h / 2)) / h
        scale = max(abs(g[j]), 1e-4)
        if abs(fd1 - fd2) > 1e-6 * scale:      # a ReLU / max-pool kink inside the stencil
            bad += 1
            continue
        checked += 1
        assert abs(fd1 - g[j]) <= 2e-6 * scale, (j, fd1, g[j])
    assert checked > 0.9 * len(idx), (bad, len(idx))


def test_finite_differences_input_gradient():
    ops, hwc, x, labels, theta = _setup(tiny_cifar, B=2)
    r = ora.microbatch(ops, hwc, theta, x, labels, want=[], want_input_grad=True)
    rng = np.random.default_rng(3)
    flat = x.reshape(-1)
    h = 1e-5
    ok = 0
    for j in rng.choice(flat.size, size=40, replace=False):
        def L(step):
            xx = flat.copy(); xx[j] += step
            return ora.microbatch(ops, hwc, theta, xx.reshape(x.shape), labels, want=[])["loss"]
        fd1 = (L(h) - L(-h)) / (2 * h)
        fd2 = (L(h / 2) - L(-h / 2)) / h
        scale = max(abs(r["dx"].reshape(-1)[j]), 1e-4)
        if abs(fd1 - fd2) > 1e-6 * scale:
            continue
        ok += 1
        assert abs(fd1 - r["dx"].reshape(-1)[j]) <= 2e-6 * scale
    assert ok >= 30


# ------------------------------------------------------------------ P2
@pytest.mark.parametrize("builder", [tiny_cifar, tiny_imagenet, tiny_v1, tiny_vgg])
def test_partition_count_invariance_bit_exact(builder):
    """Section 6.1's claim, partitioned == sequential, as a bit-exact identity:
    0, 1, 2 and 4 cuts, block-aligned and mid-block, give identical fp64 results."""
    ops, hwc, x, labels, theta = _setup(builder, B=4)
    n = len(ops)
    ref = ora.microbatch(ops, hwc, theta, x, labels)
    cut_sets = [[], [n // 2], [3, n - 1], [1, 5, 12, n - 2], wl.default_cuts(n, 4),
                [i for i in range(1, n)]]          # one op per partition
    for cuts in cut_sets:
        r = ora.microbatch(ops, hwc, theta, x, labels, cuts=cuts)
        assert r["loss"] == ref["loss"]
        assert np.array_equal(r["g"], ref["g"])
        for i in range(n):
            assert np.array_equal(r["act"][i], ref["act"][i]), (cuts, i)
            assert np.array_equal(r["dact"][i], ref["dact"][i]), (cuts, i)
        # messages: forward = the producer's activation, backward = its full gradient
        # when every consumer sits at or after the cut, else a partial sum.
        for (j, k), msg in r["fwd_msg"].items():
            t = r["live"][j][k]
            assert np.array_equal(msg, ref["act"][t])
        for (j, k), msg in r["bwd_msg"].items():
            t = r["live"][j][k]
            consumers = [i for i, o in enumerate(ops) if o.src0 == t or (o.kind == wl.ADD and o.src1 == t)]
            if min(consumers) >= cuts[j]:
                assert np.array_equal(msg, ref["dact"][t])


def test_partial_error_is_sum_over_late_consumers():
    """Mid-block cut: the shortcut tensor's partial error counts only the
    consumers at or after the cut (Eq. 7 applied per boundary tensor)."""
    ops, hwc, x, labels, theta = _setup(tiny_cifar, B=2)
    # op 0 = stem; block 1 = ops 1..8 (BN, c1, BN, c2, BN, c3, proj, ADD); cut inside it
    assert ops[7].kind == wl.CONV and ops[7].src0 == 0 and ops[8].kind == wl.ADD
    cut = 4
    r = ora.microbatch(ops, hwc, theta, x, labels, cuts=[cut])
    assert r["live"][0] == [0, 3]
    ref = ora.microbatch(ops, hwc, theta, x, labels)
    # stem output (tensor 0) is read by BN (op 1, before the cut) and the projection (op 7, after):
    w7 = theta[wl.param_offsets(ops)[0][7][0]:][:ops[7].c_out * ops[7].c_in].reshape(ops[7].c_out, 1, 1, ops[7].c_in)
    late = ora.conv_dgrad(ref["dact"][7], w7, ref["act"][0].shape, ops[7].stride, 0)
    assert np.array_equal(r["bwd_msg"][(0, 0)], late)
    assert not np.array_equal(r["bwd_msg"][(0, 0)], ref["dact"][0])


# ------------------------------------------------------------------ P3
def test_microbatch_identity():
    """g_avg = (sum_m gradient of an M=1 run on micro-batch m alone)/M; loss likewise."""
    ops, hwc, x, labels, theta = _setup(tiny_cifar, B=6)
    M = 3
    full = ora.step(ops, hwc, theta, x, labels, M, cuts=[9])
    parts = [ora.step(ops, hwc, theta, x[2 * m:2 * m + 2], labels[2 * m:2 * m + 2], 1) for m in range(M)]
    acc = np.zeros_like(full["g_avg"]); ls = 0.0
    for p in parts:
        acc += p["g_avg"]; ls += p["loss"]
    assert np.array_equal(full["g_avg"], acc / M)
    assert full["loss"] == ls / M
    for m in range(M):
        assert np.array_equal(full["g_slots"][m], parts[m]["g_avg"])
    # and it is NOT the M=1 gradient of the whole batch (BN statistics are per micro-batch)
    whole = ora.step(ops, hwc, theta, x, labels, 1)
    assert not np.allclose(whole["g_avg"], full["g_avg"], rtol=1e-9, atol=0)


def test_grad_average_ascending_sum_over_M():
    g = np.array([[1.0, 1e16], [2.0, 1.0], [3.0, -1e16]])
    out = ora.grad_average(g)
    assert out[0] == 2.0
    assert out[1] == ((1e16 + 1.0) - 1e16) / 3      # ascending order, visible in fp64 rounding


# ------------------------------------------------------------------ P4
@pytest.mark.parametrize("ks,st,pad,H", [(1, 1, 0, 6), (3, 1, 1, 6), (1, 2, 0, 6), (7, 2, 3, 12), (3, 2, 1, 7)])
def test_conv_adjoint_identities(ks, st, pad, H):
    rng = np.random.default_rng(ks * 10 + st)
    x = rng.standard_normal((2, H, H + 2, 3))
    w = rng.standard_normal((5, ks, ks, 3))
    y = ora.conv_fwd(x, w, st, pad)
    dy = rng.standard_normal(y.shape)
    lhs = np.sum(y * dy)
    assert abs(lhs - np.sum(x * ora.conv_dgrad(dy, w, x.shape, st, pad))) <= 1e-12 * abs(lhs) + 1e-12
    assert abs(lhs - np.sum(w * ora.conv_wgrad(x, dy, ks, st, pad))) <= 1e-12 * abs(lhs) + 1e-12


# ------------------------------------------------------------------ P5
@pytest.mark.parametrize("ks,st,pad", [(1, 1, 0), (3, 1, 1), (1, 2, 0), (7, 2, 3)])
def test_conv_forward_vs_im2col_brute_force(ks, st, pad):
    rng = np.random.default_rng(11)
    N, H, W, Cc, K = 2, 8, 6, 3, 4
    x = rng.standard_normal((N, H, W, Cc)); w = rng.standard_normal((K, ks, ks, Cc))
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, Cc)); xp[:, pad:pad + H, pad:pad + W] = x
    P, Q = (H + 2 * pad - ks) // st + 1, (W + 2 * pad - ks) // st + 1
    cols = np.empty((N, P, Q, ks * ks * Cc))
    for p in range(P):
        for q in range(Q):
            cols[:, p, q] = xp[:, p * st:p * st + ks, q * st:q * st + ks].reshape(N, -1)
    y = cols @ w.reshape(K, -1).T
    assert np.allclose(ora.conv_fwd(x, w, st, pad), y, rtol=1e-13, atol=1e-13)


# ------------------------------------------------------------------ P6
def test_head_closed_forms():
    rng = np.random.default_rng(5)
    for ncls in (10, 1000):
        a = rng.standard_normal((3, 2, 2, 8))
        labels = rng.integers(0, ncls, 3)
        logits, loss = ora.head_fwd(a, np.zeros((ncls, 8)), np.zeros(ncls), labels)
        assert abs(loss - np.log(ncls)) < 1e-14
        Wfc = rng.standard_normal((ncls, 8))
        logits, loss = ora.head_fwd(a, Wfc, rng.standard_normal(ncls), labels)
        dl, dW, db, da = ora.head_bwd(a, Wfc, labels, logits)
        assert np.allclose(dl.sum(axis=1), 0, atol=1e-15)
        assert abs(db.sum()) < 1e-14
    # hand-computed two-class case: pooled = 1, logits = (0, ln 3) -> p = (1/4, 3/4)
    a = np.ones((1, 2, 2, 1))
    logits, loss = ora.head_fwd(a, np.array([[0.0], [np.log(3.0)]]), np.zeros(2), [0])
    assert abs(loss - np.log(4.0)) < 1e-14
    dl, dW, db, da = ora.head_bwd(a, np.array([[0.0], [np.log(3.0)]]), [0], logits)
    assert np.allclose(dl, [[-0.75, 0.75]], atol=1e-15)
    assert np.allclose(da, 0.75 * np.log(3.0) / 4, atol=1e-15)


# ------------------------------------------------------------------ P7
def test_bn_invariants():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((4, 5, 5, 6)) * 3 + 1.5
    gamma = rng.standard_normal(6) + 2; beta = rng.standard_normal(6) + 5     # beta large: ReLU mostly open
    eps = 1e-5
    mean, var = ora.bn_stats(x)
    assert np.allclose(mean, x.reshape(-1, 6).mean(0), rtol=1e-14)
    assert np.allclose(var, x.reshape(-1, 6).var(0), rtol=1e-13)             # biased
    y = ora.bnrelu_fwd(x, gamma, beta + 100, eps) - 100                       # ReLU fully open
    assert np.allclose(y.reshape(-1, 6).mean(0), beta, atol=1e-12)
    assert np.allclose(y.reshape(-1, 6).var(0), gamma ** 2 * var / (var + eps), rtol=1e-12)
    dy = rng.standard_normal(x.shape)
    dx, dg, db = ora.bnrelu_bwd(x, dy, gamma, beta, eps)
    xh = (x - mean) / np.sqrt(var + eps)
    assert np.allclose(dx.reshape(-1, 6).sum(0), 0, atol=1e-12)
    # sum dx*xhat vanishes up to the eps term: sum xhat^2 = rows * var/(var+eps), not rows
    resid = gamma / np.sqrt(var + eps) * dg * eps / (var + eps)
    assert np.allclose((dx * xh).reshape(-1, 6).sum(0), resid, rtol=1e-6, atol=1e-12)
    assert np.all(np.abs(resid) < 1e-4)
    # ReLU mask: where the output is clamped the incoming gradient must not count
    y0 = ora.bnrelu_fwd(x, gamma, beta - 6, eps)
    dx2, dg2, db2 = ora.bnrelu_bwd(x, dy, gamma, beta - 6, eps)
    assert np.allclose(db2, (dy * (y0 > 0)).reshape(-1, 6).sum(0), rtol=1e-12)


# ------------------------------------------------------------------ P8
def test_scale_invariance_of_conv_feeding_bn():
    """A conv that feeds a BN directly: the loss does not change when its weights
    are scaled, so <w, dL/dw> = 0 up to O(eps)."""
    ops, hwc, x, labels, theta = _setup(tiny_cifar, B=4)
    g = ora.step(ops, hwc, theta, x, labels, 2)["g_avg"]
    offs, _ = wl.param_offsets(ops)
    feeds_bn = [i for i, o in enumerate(ops) if o.kind == wl.CONV
                and [c.kind for c in ops if c.src0 == i] == [wl.BNRELU]]
    assert len(feeds_bn) >= 6
    for i in feeds_bn:
        w_off, w_cnt = offs[i][0], offs[i][1]
        w, gw = theta[w_off:w_off + w_cnt], g[w_off:w_off + w_cnt]
        assert abs(np.dot(w, gw)) <= 1e-3 * np.linalg.norm(w) * np.linalg.norm(gw)


# ------------------------------------------------------------------ P9
def test_paper_two_layer_example_eq_3_to_7():
    """Fig. 'single hidden layer' with the cut between the layers: V = W1 X on
    one partition, Y' = W2 V and the loss on the other.  D2 = dL/dY' V^T,
    partial_error = W2^T dL/dY' crosses the cut, D1 = partial_error X^T."""
    rng = np.random.default_rng(2)
    d_in, d_hid, ncls, b = 3, 4, 5, 6
    ops = [wl.Op(wl.CONV, -1, -1, d_in, d_hid, 1, 1, 0, 0.0), wl.Op(wl.HEAD, 0, -1, d_hid, ncls, 0, 1, 0, 0.0)]
    X = rng.standard_normal((b, 1, 1, d_in)); labels = rng.integers(0, ncls, b)
    W1 = rng.standard_normal((d_hid, d_in)); W2 = rng.standard_normal((ncls, d_hid))
    theta = np.concatenate([W1.ravel(), W2.ravel(), np.zeros(ncls)])
    r = ora.microbatch(ops, (1, 1, d_in), theta, X, labels, cuts=[1])
    # direct evaluation, columns = samples
    Xc = X.reshape(b, d_in).T
    V = W1 @ Xc; Yp = W2 @ V
    e = np.exp(Yp - Yp.max(0)); p = e / e.sum(0)
    dYp = p.copy(); dYp[labels, np.arange(b)] -= 1; dYp /= b
    D2 = dYp @ V.T
    partial_error = W2.T @ dYp
    D1 = partial_error @ Xc.T
    assert np.allclose(r["g"][:W1.size].reshape(W1.shape), D1, rtol=1e-12, atol=1e-14)
    assert np.allclose(r["g"][W1.size:W1.size + W2.size].reshape(W2.shape), D2, rtol=1e-12, atol=1e-14)
    assert r["live"] == [[0]]
    assert np.allclose(r["bwd_msg"][(0, 0)].reshape(b, d_hid).T, partial_error, rtol=1e-12, atol=1e-14)
    assert np.allclose(r["fwd_msg"][(0, 0)].reshape(b, d_hid).T, V, rtol=1e-12, atol=1e-14)
    assert abs(r["loss"] - (-np.log(p[labels, np.arange(b)]).mean())) < 1e-13


# ------------------------------------------------------------------ P10
def _torch_step(ops, hwc, theta, x, labels, M):
    """The same step with library ops (torch CPU fp64 + autograd)."""
    import torch
    import torch.nn.functional as F
    offs, G = wl.param_offsets(ops)
    th = torch.tensor(theta, dtype=torch.float64)
    B = x.shape[0]; b = B // M
    slots, losses, acts, dacts = [], [], [], []
    for m in range(M):
        t = th.clone().requires_grad_(True)
        xin = torch.tensor(x[m * b:(m + 1) * b], dtype=torch.float64).permute(0, 3, 1, 2)
        out = []
        for o, (w_off, w_cnt, b_off, b_cnt) in zip(ops, offs):
            s0 = xin if o.src0 < 0 else out[o.src0]
            if o.kind == wl.CONV:
                w = t[w_off:w_off + w_cnt].reshape(o.c_out, o.ksize, o.ksize, o.c_in).permute(0, 3, 1, 2)
                y = F.conv2d(s0, w, stride=o.stride, padding=o.pad)
            elif o.kind == wl.BNRELU:
                y = F.relu(F.batch_norm(s0, None, None, t[w_off:w_off + w_cnt], t[b_off:b_off + b_cnt],
                                        training=True, eps=o.eps))
            elif o.kind == wl.BN:
                y = F.batch_norm(s0, None, None, t[w_off:w_off + w_cnt], t[b_off:b_off + b_cnt], training=True, eps=o.eps)
            elif o.kind == wl.RELU:
                y = F.relu(s0)
            elif o.kind == wl.ADD:
                y = s0 + out[o.src1]
            elif o.kind == wl.MAXPOOL:
                y = F.max_pool2d(s0, o.ksize, o.stride, o.pad)
            else:
                pooled = s0.mean(dim=(2, 3))
                y = pooled @ t[w_off:w_off + w_cnt].reshape(o.c_out, o.c_in).T + t[b_off:b_off + b_cnt]
            y.retain_grad()
            out.append(y)
        loss = F.cross_entropy(out[-1], torch.tensor(labels[m * b:(m + 1) * b], dtype=torch.long))
        loss.backward()
        slots.append(t.grad.numpy().copy()); losses.append(loss.item())
        acts.append([o_.detach().permute(0, 2, 3, 1).numpy() if o_.dim() == 4 else o_.detach().numpy() for o_ in out])
        dacts.append([o_.grad.permute(0, 2, 3, 1).numpy() if o_.dim() == 4 else o_.grad.numpy() for o_ in out])
    return np.array(slots), np.array(losses), acts, dacts


@pytest.mark.parametrize("builder,B,M", [(tiny_cifar, 4, 2), (tiny_imagenet, 4, 2), (tiny_v1, 4, 2), (tiny_vgg, 4, 2)])
def test_against_torch_autograd_small(builder, B, M):
    ops, hwc, x, labels, theta = _setup(builder, B=B, seed=1)
    slots, losses, acts, dacts = _torch_step(ops, hwc, theta, x, labels, M)
    r = ora.step(ops, hwc, theta, x, labels, M, cuts=[len(ops) // 2])
    assert np.allclose(r["losses"], losses, rtol=1e-12)
    assert np.allclose(r["g_slots"], slots, rtol=1e-8, atol=1e-11)
    assert np.allclose(r["g_avg"], slots.sum(0) / M, rtol=1e-8, atol=1e-11)
    b = B // M
    mb = ora.microbatch(ops, hwc, theta, x[:b], labels[:b])
    for i in range(len(ops)):
        assert np.allclose(mb["act"][i].reshape(acts[0][i].shape), acts[0][i], rtol=1e-9, atol=1e-11), i
        assert np.allclose(mb["dact"][i].reshape(dacts[0][i].shape), dacts[0][i], rtol=1e-8, atol=1e-12), i


def test_against_torch_autograd_config1():
    """Benchmark configuration 1 end to end (ResNet-11, 8x3x32x32, 2 partitions x 2 micro-batches)."""
    c = wl.config("r11")
    x, labels = wl.draw_inputs(c["B"], c["in_hwc"], 10)
    theta = wl.draw_params(c["ops"])
    slots, losses, _, _ = _torch_step(c["ops"], c["in_hwc"], theta.astype(np.float64), x.astype(np.float64), labels, c["M"])
    r = ora.step(c["ops"], c["in_hwc"], theta, x, labels, c["M"], cuts=c["cuts"])
    assert np.allclose(r["losses"], losses, rtol=1e-12)
    assert np.allclose(r["g_avg"], slots.sum(0) / c["M"], rtol=1e-8, atol=1e-11)


def test_against_torch_autograd_resnet110_reduced_batch():
    """Configuration 3's network (ResNet-110 v2, 4 partitions x 4 micro-batches) at batch 8."""
    c = wl.config("r110")
    x, labels = wl.draw_inputs(8, c["in_hwc"], 10)
    theta = wl.draw_params(c["ops"])
    slots, losses, _, _ = _torch_step(c["ops"], c["in_hwc"], theta.astype(np.float64), x.astype(np.float64), labels, 4)
    r = ora.step(c["ops"], c["in_hwc"], theta, x, labels, 4, cuts=c["cuts"])
    assert np.allclose(r["losses"], losses, rtol=1e-11)
    num = np.linalg.norm(r["g_avg"] - slots.sum(0) / 4); den = np.linalg.norm(slots.sum(0) / 4)
    assert num <= 1e-8 * den


# ------------------------------------------------------------------ max-pool
def test_maxpool_against_brute_force_and_tie_rule():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 7, 7, 3))
    y = ora.maxpool_fwd(x, 3, 2, 1)
    xp = np.full((2, 9, 9, 3), -np.inf); xp[:, 1:8, 1:8] = x
    for p in range(4):
        for q in range(4):
            assert np.array_equal(y[:, p, q], xp[:, 2 * p:2 * p + 3, 2 * q:2 * q + 3].max(axis=(1, 2)))
    # ties: constant input -> the first window position inside the image gets the gradient
    x1 = np.ones((1, 4, 4, 1)); dy = np.arange(1, 5, dtype=np.float64).reshape(1, 2, 2, 1)
    dx = ora.maxpool_bwd(x1, dy, 3, 2, 1)
    exp = np.zeros((4, 4)); exp[0, 0] = 1; exp[0, 1] = 2; exp[1, 0] = 3; exp[1, 1] = 4
    assert np.array_equal(dx[0, :, :, 0], exp)


# ------------------------------------------------------------------ ReLU decisions
def test_supplied_relu_decisions_window():
    """Decisions of another implementation are honoured only inside |z| < tau*|gamma|, and a
    gradient evaluated with a flipped in-window decision equals the plain gradient of a nearby
    problem whose own decision is the flipped one (here: beta nudged across the kink)."""
    ops, hwc, x, labels, theta = _setup(tiny_cifar, B=4)
    plain = ora.microbatch(ops, hwc, theta, x, labels)
    bn = [i for i, o in enumerate(ops) if o.kind == wl.BNRELU]
    offs, _ = wl.param_offsets(ops)
    own = {i: (plain["act"][i] > 0).astype(np.uint8) for i in bn}
    # own decisions, any tau: bit-identical, nothing used, no violation
    same = ora.microbatch(ops, hwc, theta, x, labels, decisions=own, tau=0.05)
    assert np.array_equal(same["g"], plain["g"]) and same["decisions_used"] == 0 and same["decision_violations"] == 0
    # all decisions inverted with tau = 0: every one is a violation, none is used
    inv = {i: 1 - d for i, d in own.items()}
    r = ora.microbatch(ops, hwc, theta, x, labels, decisions=inv, tau=0.0)
    assert np.array_equal(r["g"], plain["g"]) and r["decisions_used"] == 0
    assert r["decision_violations"] == sum(d.size for d in own.values())
    # flip the decision of the element of one BN whose pre-activation is closest to zero
    i = bn[2]
    src = ops[i].src0
    xin = plain["act"][src]; C = xin.shape[-1]
    gamma = theta[offs[i][0]:offs[i][0] + C]; beta = theta[offs[i][2]:offs[i][2] + C]
    mean, var = ora.bn_stats(xin)
    z = gamma * (xin - mean) / np.sqrt(var + ops[i].eps) + beta
    flat = np.abs(z / gamma).reshape(-1, C)
    row, ch = np.unravel_index(np.argmin(flat), flat.shape)
    zmin = z.reshape(-1, C)[row, ch]
    flipped = {k: v.copy() for k, v in own.items()}
    flipped[i].reshape(-1, C)[row, ch] ^= 1
    two = np.sort(flat.ravel())[:2]
    tau = 0.5 * (two[0] + two[1])
    assert np.sum(np.abs(z / gamma) < tau) == 1                      # only that element is undecided
    r = ora.microbatch(ops, hwc, theta, x, labels, decisions=flipped, tau=tau)
    assert r["decisions_used"] == 1 and r["decision_violations"] == 0
    assert not np.array_equal(r["g"], plain["g"])
    # the nearby problem: beta_ch moved by 2*|z| so that its own decision flips
    theta2 = theta.copy()
    theta2[offs[i][2] + ch] -= 2.0 * zmin
    near = ora.microbatch(ops, hwc, theta2, x, labels)
    assert (near["act"][i] > 0).reshape(-1, C)[row, ch] != (plain["act"][i] > 0).reshape(-1, C)[row, ch]
    d_flip = np.linalg.norm(r["g"] - near["g"]); d_plain = np.linalg.norm(plain["g"] - near["g"])
    assert d_flip < 0.05 * d_plain, (d_flip, d_plain)                # the flip explains the jump
    # partition-by-partition execution honours the decisions identically
    rp = ora.microbatch(ops, hwc, theta, x, labels, cuts=[4, 13], decisions=flipped, tau=tau)
    assert np.array_equal(rp["g"], r["g"]) and rp["decisions_used"] == 1


def test_supplied_decisions_of_a_stand_alone_relu():
    """The same rule for the RELU op of the post-activation block: the window is |x| < tau on the op's input, an
    in-window flip changes exactly that element's gate (dx = dy there instead of 0, or the reverse)."""
    ops, hwc, x, labels, theta = _setup(tiny_v1, B=4)
    plain = ora.microbatch(ops, hwc, theta, x, labels)
    relus = [i for i, o in enumerate(ops) if o.kind == wl.RELU]
    assert relus
    own = {i: (plain["act"][ops[i].src0] > 0).astype(np.uint8) for i in relus}
    same = ora.microbatch(ops, hwc, theta, x, labels, decisions=own, tau=0.1)
    assert np.array_equal(same["g"], plain["g"]) and same["decisions_used"] == 0 and same["decision_violations"] == 0
    inv = {i: 1 - d for i, d in own.items()}
    r = ora.microbatch(ops, hwc, theta, x, labels, decisions=inv, tau=0.0)
    assert np.array_equal(r["g"], plain["g"]) and r["decision_violations"] == sum(d.size for d in own.values())
    i = relus[-1]
    xin = plain["act"][ops[i].src0]
    flat = np.abs(xin).ravel()
    j = int(np.argmin(flat))
    two = np.sort(flat)[:2]
    tau = 0.5 * (two[0] + two[1])
    flipped = {k: v.copy() for k, v in own.items()}
    flipped[i].reshape(-1)[j] ^= 1
    r = ora.microbatch(ops, hwc, theta, x, labels, decisions=flipped, tau=tau)
    assert r["decisions_used"] == 1 and r["decision_violations"] == 0
    d_plain, d_flip, dy = plain["dact"][ops[i].src0].ravel(), r["dact"][ops[i].src0].ravel(), plain["dact"][i].ravel()
    # the op's input has the RELU as its only reader here, so its gradient is the gated dy
    if len([o for o in ops if o.src0 == ops[i].src0 or o.src1 == ops[i].src0]) == 1:
        assert d_flip[j] == (dy[j] if flipped[i].reshape(-1)[j] else 0.0)
        assert np.array_equal(np.delete(d_flip, j), np.delete(d_plain, j))


# ---------------------------------------------------------------- parameter update (Section 5.3, apply_gradients)
def test_sgd_momentum_closed_forms():
    """Constant gradient g, no decay: v_k = -lr*g*(1-mu^k)/(1-mu) and theta_k = theta_0 + sum_i v_i (geometric sums);
    mu = 0 is plain descent; with decay and mu = 0 on a zero gradient theta shrinks by (1 - lr*wd) per step."""
    rng = np.random.default_rng(7)
    G, lr, mu = 37, 0.1, 0.9
    theta0, g = rng.standard_normal(G), rng.standard_normal(G)
    theta, v = theta0.copy(), np.zeros(G)
    for k in range(1, 6):
        theta, v = ora.sgd_momentum(theta, v, g, lr, mu)
        vk = -lr * g * (1 - mu ** k) / (1 - mu)
        sum_v = -lr * g * (k - mu * (1 - mu ** k) / (1 - mu)) / (1 - mu)
        np.testing.assert_allclose(v, vk, rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(theta, theta0 + sum_v, rtol=1e-13, atol=1e-15)
    t1, v1 = ora.sgd_momentum(theta0, np.zeros(G), g, lr)
    np.testing.assert_allclose(t1, theta0 - lr * g, rtol=1e-15)
    np.testing.assert_allclose(v1, -lr * g, rtol=1e-15)
    t, v = theta0.copy(), np.zeros(G)
    for _ in range(4):
        t, v = ora.sgd_momentum(t, v, np.zeros(G), lr, 0.0, 0.5)
    np.testing.assert_allclose(t, theta0 * (1 - lr * 0.5) ** 4, rtol=1e-14)
    # sign: a step along -g lowers a quadratic 0.5*|theta|^2 whose gradient is theta
    t2, _ = ora.sgd_momentum(theta0, np.zeros(G), theta0, 0.3)
    assert np.sum(t2 ** 2) < np.sum(theta0 ** 2)
    # the inputs are not modified
    assert np.array_equal(g, g.copy()) and not np.shares_memory(t1, theta0)


def test_sgd_step_lowers_the_loss_of_a_tiny_net():
    """Descent property on the real objective: for a small enough rate, L(theta - lr*g) < L(theta)."""
    ops, hwc = wl.resnet_v2_cifar(1, (4, 8, 16), 3), (8, 8, 3)
    x, labels = wl.draw_inputs(4, hwc, 3)
    theta = wl.draw_params(ops, bn_jitter=0.2)
    r0 = ora.step(ops, hwc, theta, x, labels, 2)
    theta1, _ = ora.sgd_momentum(theta, np.zeros(theta.size), r0["g_avg"], 0.05)
    r1 = ora.step(ops, hwc, theta1, x, labels, 2)
    assert r1["loss"] < r0["loss"]
