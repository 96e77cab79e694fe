"""Seeded synthetic inputs: images ~ N(0,1), uniform labels, He-normal weights.

Stand-ins for CIFAR-10 (32x32x3) and for 224x224x3 images.  numpy PCG64;
fp64 draws rounded to fp32; seeds: images 1911, labels 5146, parameters 2020.
Parameters are drawn op by op in flat-buffer order: conv weights
[c_out][r][s][c_in] ~ N(0, 2/fan_in) with fan_in = c_in*r*s, BN gamma = 1 and
beta = 0, FC weights ~ N(0, 2/C) and FC bias = 0.
"""
import numpy as np

from .resnet_spec import CONV, BNRELU, BN, HEAD, MAXPOOL

SEED_X, SEED_LABELS, SEED_PARAMS = 1911, 5146, 2020


def tensor_shapes(ops, in_hwc):
    """(H, W, C) of every op's output (the head's output is (1, 1, classes))."""
    out = []
    for o in ops:
        H, W, C = in_hwc if o.src0 < 0 else out[o.src0]
        if o.kind in (CONV, MAXPOOL):
            out.append(((H + 2 * o.pad - o.ksize) // o.stride + 1, (W + 2 * o.pad - o.ksize) // o.stride + 1, o.c_out))
        elif o.kind == HEAD:
            out.append((1, 1, o.c_out))
        else:
            out.append((H, W, C))
    return out


def param_offsets(ops):
    """[(w_off, w_cnt, b_off, b_cnt)] per op and the total count."""
    at, out = 0, []
    for o in ops:
        wc = bc = 0
        if o.kind == CONV:
            wc = o.c_out * o.ksize * o.ksize * o.c_in
        elif o.kind in (BNRELU, BN):
            wc = bc = o.c_in
        elif o.kind == HEAD:
            wc, bc = o.c_out * o.c_in, o.c_out
        out.append((at, wc, at + wc, bc))
        at += wc + bc
    return out, at


def draw_inputs(B, in_hwc, n_classes, seed_x=SEED_X, seed_labels=SEED_LABELS):
    x = np.random.Generator(np.random.PCG64(seed_x)).standard_normal((B,) + tuple(in_hwc)).astype(np.float32)
    labels = np.random.Generator(np.random.PCG64(seed_labels)).integers(0, n_classes, size=B).astype(np.int32)
    return x, labels


def draw_params(ops, seed=SEED_PARAMS, bn_jitter=0.0):
    """Flat fp32 parameter vector.  bn_jitter > 0 perturbs gamma/beta (tests only),
    so that BN gradients are exercised away from the gamma=1, beta=0 point."""
    rng = np.random.Generator(np.random.PCG64(seed))
    offs, G = param_offsets(ops)
    theta = np.zeros(G, dtype=np.float32)
    for o, (w_off, w_cnt, b_off, b_cnt) in zip(ops, offs):
        if o.kind == CONV:
            fan_in = o.c_in * o.ksize * o.ksize
            theta[w_off:w_off + w_cnt] = (rng.standard_normal(w_cnt) * np.sqrt(2.0 / fan_in)).astype(np.float32)
        elif o.kind in (BNRELU, BN):
            theta[w_off:w_off + w_cnt] = 1.0
            if bn_jitter:
                theta[w_off:w_off + w_cnt] += (bn_jitter * rng.standard_normal(w_cnt)).astype(np.float32)
                theta[b_off:b_off + b_cnt] = (bn_jitter * rng.standard_normal(b_cnt)).astype(np.float32)
        elif o.kind == HEAD:
            theta[w_off:w_off + w_cnt] = (rng.standard_normal(w_cnt) * np.sqrt(2.0 / o.c_in)).astype(np.float32)
    return theta
