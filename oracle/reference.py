"""ctypes front end of the fp64 CPU oracle.  TEST INFRASTRUCTURE, not the product.

Only tests, the smoke entry and the benchmark's CPU-baseline leg may import
this module.  It imports nothing from the CUDA package.  Ops are plain tuples
``(kind, src0, src1, c_in, c_out, ksize, stride, pad, eps)`` with the kind codes
below; tensors are numpy arrays, channels innermost ([n][h][w][c]); fp32 inputs
are widened to fp64 (exactly) before the C code sees them.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

CONV, BNRELU, ADD, MAXPOOL, HEAD, BN, RELU = 1, 2, 3, 4, 5, 6, 7


class _Op(C.Structure):
    _fields_ = [("kind", C.c_int32), ("src0", C.c_int32), ("src1", C.c_int32),
                ("c_in", C.c_int32), ("c_out", C.c_int32), ("ksize", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32), ("eps", C.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
    return _lib


def _ops(ops):
    arr = (_Op * len(ops))()
    for i, o in enumerate(ops):
        k, s0, s1, ci, co, ks, st, pd, eps = o
        arr[i] = _Op(int(k), int(s0), int(s1), int(ci), int(co), int(ks), int(st), int(pd), float(eps))
    return arr


def _i32(seq):
    return (C.c_int32 * len(seq))(*[int(v) for v in seq])


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(C.POINTER(C.c_double))


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with status {rc}")


# ---------------------------------------------------------------- bookkeeping
def shapes(ops, in_hwc):
    out = (C.c_int32 * (3 * len(ops)))()
    _check(lib().ora_shapes(_ops(ops), len(ops), _i32(in_hwc), out), "shapes")
    return [tuple(out[3 * i:3 * i + 3]) for i in range(len(ops))]


def param_layout(ops):
    n = len(ops)
    arrs = [(C.c_int64 * n)() for _ in range(4)]
    total = C.c_int64()
    _check(lib().ora_param_layout(_ops(ops), n, *arrs, C.byref(total)), "param_layout")
    w_off, w_cnt, b_off, b_cnt = [list(a) for a in arrs]
    return w_off, w_cnt, b_off, b_cnt, total.value


def partition_of_ops(n_ops, cuts):
    out = (C.c_int32 * n_ops)()
    _check(lib().ora_partition_of_ops(n_ops, _i32(cuts), len(cuts), out), "partition_of_ops")
    return list(out)


def live_set(ops, cut):
    out = (C.c_int32 * len(ops))()
    cnt = C.c_int32()
    _check(lib().ora_live_set(_ops(ops), len(ops), int(cut), out, C.byref(cnt)), "live_set")
    return list(out[:cnt.value])


def microbatch_range(B, M, m):
    a, b = C.c_int32(), C.c_int32()
    _check(lib().ora_microbatch_range(B, M, m, C.byref(a), C.byref(b)), "microbatch_range")
    return a.value, b.value


def schedule_tick(P, M, p, m):
    a, b = C.c_int32(), C.c_int32()
    _check(lib().ora_schedule_tick(P, M, p, m, C.byref(a), C.byref(b)), "schedule_tick")
    return a.value, b.value


# ---------------------------------------------------------------- single ops
def _out_hw(H, W, R, st, pad):
    return (H + 2 * pad - R) // st + 1, (W + 2 * pad - R) // st + 1


def conv_fwd(x, w, stride, pad):
    N, H, W, Cc = x.shape
    K, R = w.shape[0], w.shape[1]
    P, Q = _out_hw(H, W, R, stride, pad)
    y = np.empty((N, P, Q, K))
    xa, xp = _d(x); wa, wp = _d(w)
    lib().ora_conv_fwd(xp, N, H, W, Cc, wp, K, R, stride, pad, y.ctypes.data_as(C.POINTER(C.c_double)))
    return y


def conv_dgrad(dy, w, x_shape, stride, pad):
    N, H, W, Cc = x_shape
    K, R = w.shape[0], w.shape[1]
    dx = np.empty(x_shape)
    da, dp = _d(dy); wa, wp = _d(w)
    lib().ora_conv_dgrad(dp, N, H, W, Cc, wp, K, R, stride, pad, dx.ctypes.data_as(C.POINTER(C.c_double)))
    return dx


def conv_wgrad(x, dy, ksize, stride, pad):
    N, H, W, Cc = x.shape
    K = dy.shape[3]
    dw = np.empty((K, ksize, ksize, Cc))
    xa, xp = _d(x); da, dp = _d(dy)
    lib().ora_conv_wgrad(xp, N, H, W, Cc, dp, K, ksize, stride, pad, dw.ctypes.data_as(C.POINTER(C.c_double)))
    return dw


def bn_stats(x):
    Cc = x.shape[-1]
    rows = x.size // Cc
    mean, var = np.empty(Cc), np.empty(Cc)
    xa, xp = _d(x)
    lib().ora_bn_stats(xp, C.c_int64(rows), Cc, mean.ctypes.data_as(C.POINTER(C.c_double)),
                       var.ctypes.data_as(C.POINTER(C.c_double)))
    return mean, var


def bnrelu_fwd(x, gamma, beta, eps):
    Cc = x.shape[-1]
    rows = x.size // Cc
    y = np.empty(x.shape)
    xa, xp = _d(x); ga, gp = _d(gamma); ba, bp = _d(beta)
    lib().ora_bnrelu_fwd(xp, C.c_int64(rows), Cc, gp, bp, C.c_double(eps), y.ctypes.data_as(C.POINTER(C.c_double)))
    return y


def bnrelu_bwd(x, dy, gamma, beta, eps):
    Cc = x.shape[-1]
    rows = x.size // Cc
    dx, dg, db = np.empty(x.shape), np.empty(Cc), np.empty(Cc)
    xa, xp = _d(x); da, dp = _d(dy); ga, gp = _d(gamma); ba, bp = _d(beta)
    P = C.POINTER(C.c_double)
    lib().ora_bnrelu_bwd(xp, dp, C.c_int64(rows), Cc, gp, bp, C.c_double(eps),
                         dx.ctypes.data_as(P), dg.ctypes.data_as(P), db.ctypes.data_as(P))
    return dx, dg, db


def maxpool_fwd(x, ksize, stride, pad):
    N, H, W, Cc = x.shape
    P, Q = _out_hw(H, W, ksize, stride, pad)
    y = np.empty((N, P, Q, Cc))
    xa, xp = _d(x)
    lib().ora_maxpool_fwd(xp, N, H, W, Cc, ksize, stride, pad, y.ctypes.data_as(C.POINTER(C.c_double)))
    return y


def maxpool_bwd(x, dy, ksize, stride, pad):
    N, H, W, Cc = x.shape
    dx = np.empty(x.shape)
    xa, xp = _d(x); da, dp = _d(dy)
    lib().ora_maxpool_bwd(xp, dp, N, H, W, Cc, ksize, stride, pad, dx.ctypes.data_as(C.POINTER(C.c_double)))
    return dx


def head_fwd(a, Wfc, bias, labels):
    b, H, W, Cc = a.shape
    ncls = Wfc.shape[0]
    logits = np.empty((b, ncls))
    loss = C.c_double()
    aa, ap = _d(a); wa, wp = _d(Wfc); ba, bp = _d(bias)
    lib().ora_head_fwd(ap, b, H, W, Cc, wp, bp, ncls, _i32(labels),
                       logits.ctypes.data_as(C.POINTER(C.c_double)), C.byref(loss))
    return logits, loss.value


def head_bwd(a, Wfc, labels, logits):
    b, H, W, Cc = a.shape
    ncls = Wfc.shape[0]
    dlogits, dW, dbias, da = np.empty((b, ncls)), np.empty((ncls, Cc)), np.empty(ncls), np.empty(a.shape)
    aa, ap = _d(a); wa, wp = _d(Wfc); la, lp = _d(logits)
    P = C.POINTER(C.c_double)
    lib().ora_head_bwd(ap, b, H, W, Cc, wp, ncls, _i32(labels), lp, dlogits.ctypes.data_as(P),
                       dW.ctypes.data_as(P), dbias.ctypes.data_as(P), da.ctypes.data_as(P))
    return dlogits, dW, dbias, da


def grad_average(g_slots):
    g_slots = np.ascontiguousarray(g_slots, dtype=np.float64)
    M, G = g_slots.shape
    out = np.empty(G)
    lib().ora_grad_average(g_slots.ctypes.data_as(C.POINTER(C.c_double)), M, C.c_int64(G),
                           out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def sgd_momentum(theta, v, g, lr, momentum=0.0, weight_decay=0.0):
    """Returns (theta', v') of one Keras-form SGD step (Section 5.3, apply_gradients); inputs are not modified."""
    theta = np.array(theta, dtype=np.float64); v = np.array(v, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    P = C.POINTER(C.c_double)
    lib().ora_sgd_momentum(theta.ctypes.data_as(P), v.ctypes.data_as(P), g.ctypes.data_as(P), C.c_int64(theta.size),
                           C.c_double(lr), C.c_double(momentum), C.c_double(weight_decay))
    return theta, v


# ---------------------------------------------------------------- sweeps
def _ptr_array(bufs):
    arr = (C.POINTER(C.c_double) * len(bufs))()
    for i, b in enumerate(bufs):
        arr[i] = b.ctypes.data_as(C.POINTER(C.c_double)) if b is not None else None
    return arr


def _decision_array(n, decisions):
    arr = (C.POINTER(C.c_uint8) * n)()
    keep = []
    for i, d in decisions.items():
        d = np.ascontiguousarray(d, dtype=np.uint8)
        keep.append(d)
        arr[i] = d.ctypes.data_as(C.POINTER(C.c_uint8))
    return arr, keep


def microbatch(ops, in_hwc, theta, x, labels, cuts=None, want=None, want_input_grad=False, decisions=None, tau=0.0):
    """One micro-batch.  Returns a dict with loss, g, act{op}, dact{op} and, when
    ``cuts`` is given (partition-by-partition execution), fwd_msg / bwd_msg
    keyed by (cut index, position in the live set).  ``want`` limits which ops'
    tensors are kept (default: all).  ``decisions`` maps a BNRELU (or RELU) op to the
    (z > 0) decisions of another implementation, honoured inside the window
    |z| < tau*|gamma| (RELU: |x| < tau); the result then carries decisions_used / decision_violations."""
    n = len(ops)
    b = x.shape[0]
    shp = shapes(ops, in_hwc)
    G = param_layout(ops)[4]
    ta, tp = _d(theta)
    xa, xp = _d(x)
    if ta.size != G:
        raise ValueError("parameter vector has the wrong length")
    want = set(range(n)) if want is None else set(want)
    act = [np.empty((b,) + shp[i]) if i in want else None for i in range(n)]
    dact = [np.empty((b,) + shp[i]) if i in want else None for i in range(n)]
    g = np.empty(G)
    loss = C.c_double()
    gp = g.ctypes.data_as(C.POINTER(C.c_double))
    res = {}
    dec, dec_keep = _decision_array(n, decisions) if decisions else (None, None)
    counts = (C.c_int64 * 2)(0, 0)
    if cuts is None:
        dx = np.empty(x.shape) if want_input_grad else None
        rc = lib().ora_microbatch_dec(_ops(ops), n, b, _i32(in_hwc), tp, xp, _i32(labels),
                                  dec, C.c_double(tau), counts,
                                  _ptr_array(act), _ptr_array(dact),
                                  dx.ctypes.data_as(C.POINTER(C.c_double)) if dx is not None else None,
                                  gp, C.byref(loss))
        _check(rc, "microbatch")
        if dx is not None:
            res["dx"] = dx
    else:
        lives = [live_set(ops, c) for c in cuts]
        max_live = max([len(l) for l in lives] + [1])
        fwd = [[np.empty((b,) + shp[t]) for t in l] + [None] * (max_live - len(l)) for l in lives]
        bwd = [[np.empty((b,) + shp[t]) for t in l] + [None] * (max_live - len(l)) for l in lives]
        flat_f = [m for row in fwd for m in row] or [None]
        flat_b = [m for row in bwd for m in row] or [None]
        rc = lib().ora_microbatch_partitioned_dec(_ops(ops), n, b, _i32(in_hwc), _i32(cuts), len(cuts), max_live,
                                              tp, xp, _i32(labels), dec, C.c_double(tau), counts,
                                              _ptr_array(act), _ptr_array(dact),
                                              _ptr_array(flat_f), _ptr_array(flat_b), gp, C.byref(loss))
        _check(rc, "microbatch_partitioned")
        res["live"] = lives
        res["fwd_msg"] = {(j, i): fwd[j][i] for j, l in enumerate(lives) for i in range(len(l))}
        res["bwd_msg"] = {(j, i): bwd[j][i] for j, l in enumerate(lives) for i in range(len(l))}
    res.update(decisions_used=counts[0], decision_violations=counts[1])
    res.update(loss=loss.value, g=g,
               act={i: a for i, a in enumerate(act) if a is not None},
               dact={i: a for i, a in enumerate(dact) if a is not None})
    return res


def step(ops, in_hwc, theta, x, labels, M, cuts=None):
    """The whole step: per-micro-batch gradient slots, their average, the losses."""
    n = len(ops)
    B = x.shape[0]
    G = param_layout(ops)[4]
    ta, tp = _d(theta)
    xa, xp = _d(x)
    g_slots, g_avg, losses = np.empty((M, G)), np.empty(G), np.empty(M)
    loss = C.c_double()
    P = C.POINTER(C.c_double)
    rc = lib().ora_step(_ops(ops), n, B, _i32(in_hwc), _i32(cuts or []), len(cuts) if cuts is not None else -1, M,
                        tp, xp, _i32(labels), g_slots.ctypes.data_as(P), g_avg.ctypes.data_as(P),
                        losses.ctypes.data_as(P), C.byref(loss))
    _check(rc, "step")
    return dict(g_slots=g_slots, g_avg=g_avg, losses=losses, loss=loss.value)
